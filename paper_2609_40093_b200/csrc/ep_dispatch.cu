// ep_dispatch / ep_group: row movers. One bf16 row is H/8 16-byte vectors; a group of
// G threads (G = 32, 64 or 128, chosen from the row length) owns one source row,
// loads up to kVecPerThread vectors per thread into registers once, and stores
// them to every destination row. Each warp finds its row's distinct destinations
// by itself (K <= 32 slots, one per lane, duplicates dropped with a warp match),
// so there is no shared memory and no block-wide barrier.
#include "ep_common.cuh"

namespace ep {
namespace {

constexpr int kBlock = 128;
constexpr int kVecPerThread = 8;

__device__ __forceinline__ void flag_status(int32_t *status, int bits)
{
    if (status) atomicOr(status, bits);
}

// recv[recv_slot[t][k]] = x[t] for the distinct slots of token t.
template <int G>
__global__ void __launch_bounds__(kBlock)
dispatch_rows_kernel(const uint4 *__restrict__ x, const int32_t *__restrict__ recv_slot, uint4 *recv,
                     int T, int K, int vec_per_row, long long capacity_rows, int32_t *status)
{
    const int lane = threadIdx.x & 31;
    const int g = threadIdx.x % G;                       // position inside the row group
    const int t = blockIdx.x * (kBlock / G) + threadIdx.x / G;
    if (t >= T) return;                                   // whole warps leave together (G >= 32)

    int32_t slot = lane < K ? __ldg(recv_slot + (size_t)t * K + lane) : -1;
    if (slot >= capacity_rows) {
        flag_status(status, EP_STATUS_CAPACITY);
        slot = -1;
    }
    // the k's of a token that land on one rank share a slot: keep the lowest k
    const unsigned same = __match_any_sync(kFullMask, slot);
    unsigned todo = __ballot_sync(kFullMask, slot >= 0 && (same & lanemask_lt()) == 0);

    const uint4 *src = x + (size_t)t * vec_per_row;
    for (int base = 0; base < vec_per_row; base += G * kVecPerThread) {  // trip count uniform over the warp
        const int v0 = base + g;
        uint4 buf[kVecPerThread];
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) buf[u] = ld_stream(src + v);
        }
        for (unsigned m = todo; m; m &= m - 1) {
            const int32_t row = __shfl_sync(kFullMask, slot, __ffs(m) - 1);
            uint4 *dst = recv + (size_t)row * vec_per_row;
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) {
                const int v = v0 + u * G;
                if (v < vec_per_row) st_stream(dst + v, buf[u]);
            }
        }
    }
}

// grouped[p] = recv[pair_row[p]] for p < P = *n_pairs.
template <int G>
__global__ void __launch_bounds__(kBlock)
group_rows_kernel(const uint4 *__restrict__ recv, long long recv_rows, const int32_t *__restrict__ pair_row,
                  const int32_t *__restrict__ n_pairs, uint4 *grouped, long long capacity_rows,
                  int vec_per_row, int32_t *status)
{
    const int g = threadIdx.x % G;
    const long long p = (long long)blockIdx.x * (kBlock / G) + threadIdx.x / G;
    if (p >= __ldg(n_pairs)) return;
    if (p >= capacity_rows) {
        if (g == 0) flag_status(status, EP_STATUS_CAPACITY);
        return;
    }
    const int32_t row = __ldg(pair_row + p);
    if (row < 0 || row >= recv_rows) {
        if (g == 0) flag_status(status, EP_STATUS_CAPACITY);
        return;
    }
    const uint4 *src = recv + (size_t)row * vec_per_row;
    uint4 *dst = grouped + (size_t)p * vec_per_row;
    for (int v0 = g; v0 < vec_per_row; v0 += G * kVecPerThread) {
        uint4 buf[kVecPerThread];
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) buf[u] = ld_stream(src + v);
        }
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) st_stream(dst + v, buf[u]);
        }
    }
}

int pick_group(int vec_per_row)
{
    if (vec_per_row <= 32 * kVecPerThread) return 32;
    if (vec_per_row <= 64 * kVecPerThread) return 64;
    return 128;
}

}  // namespace

int launch_dispatch(const ep_shape_t &s, const void *x, const int32_t *recv_slot, void *recv,
                    int64_t capacity_rows, int32_t *status, cudaStream_t stream)
{
    const int T = s.num_tokens, K = s.top_k, vpr = s.hidden / 8;
    const uint4 *xs = static_cast<const uint4 *>(x);
    uint4 *rd = static_cast<uint4 *>(recv);
    switch (pick_group(vpr)) {
    case 32:
        dispatch_rows_kernel<32><<<ceil_div(T, kBlock / 32), kBlock, 0, stream>>>(xs, recv_slot, rd, T, K, vpr, capacity_rows, status);
        break;
    case 64:
        dispatch_rows_kernel<64><<<ceil_div(T, kBlock / 64), kBlock, 0, stream>>>(xs, recv_slot, rd, T, K, vpr, capacity_rows, status);
        break;
    default:
        dispatch_rows_kernel<128><<<T, kBlock, 0, stream>>>(xs, recv_slot, rd, T, K, vpr, capacity_rows, status);
    }
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

int launch_group(const ep_shape_t &s, const void *recv, int64_t recv_rows, const int32_t *pair_row,
                 const int32_t *n_pairs, void *grouped, int64_t capacity_rows, int32_t *status,
                 cudaStream_t stream)
{
    const long long max_pairs = (long long)s.num_tokens * s.top_k;
    const int vpr = s.hidden / 8;
    const uint4 *rs = static_cast<const uint4 *>(recv);
    uint4 *gd = static_cast<uint4 *>(grouped);
    switch (pick_group(vpr)) {
    case 32:
        group_rows_kernel<32><<<(unsigned)((max_pairs + 3) / 4), kBlock, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, status);
        break;
    case 64:
        group_rows_kernel<64><<<(unsigned)((max_pairs + 1) / 2), kBlock, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, status);
        break;
    default:
        group_rows_kernel<128><<<(unsigned)max_pairs, kBlock, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, status);
    }
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

}  // namespace ep

extern "C" int ep_dispatch(const ep_shape_t *shape, const void *x, const int32_t *recv_slot, void *recv,
                           int64_t recv_capacity_rows, int32_t *status, void *stream)
{
    int rc = ep::check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x || !recv_slot || !recv) return EP_ERR_NULL;
    if (!ep::aligned16(x) || !ep::aligned16(recv) || recv_capacity_rows < 0) return EP_ERR_INVALID_ARG;
    return ep::launch_dispatch(*shape, x, recv_slot, recv, recv_capacity_rows, status, static_cast<cudaStream_t>(stream));
}

extern "C" int ep_group(const ep_shape_t *shape, const void *recv, int64_t recv_rows, const int32_t *pair_row,
                        const int32_t *expert_offsets, void *grouped, int64_t grouped_capacity_rows,
                        int32_t *status, void *stream)
{
    int rc = ep::check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!recv || !pair_row || !expert_offsets || !grouped) return EP_ERR_NULL;
    if (!ep::aligned16(recv) || !ep::aligned16(grouped) || recv_rows < 0 || grouped_capacity_rows < 0)
        return EP_ERR_INVALID_ARG;
    return ep::launch_group(*shape, recv, recv_rows, pair_row, expert_offsets + shape->num_experts, grouped,
                            grouped_capacity_rows, status, static_cast<cudaStream_t>(stream));
}
