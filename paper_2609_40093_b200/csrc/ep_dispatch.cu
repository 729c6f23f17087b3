// ep_dispatch / ep_group: row movers. One bf16 row is H/8 16-byte vectors; a group of
// G threads (a multiple of 32, chosen from the row length) owns one source row,
// loads U vectors per thread into registers once, and stores them to every
// destination row. Each warp finds its row's distinct destinations by itself
// (K <= 32 slots, one per lane, duplicates dropped with a warp match), so there
// is no shared memory and no block-wide barrier.
#include "ep_common.cuh"

namespace ep {
namespace {

constexpr int kMinBlock = 128;

// Thread group per row and vectors per thread: G*U covers the row when it can
// (long rows: many threads with one or two vectors each; short rows: one warp).
struct RowPlan {
    int G, U, block, rows_per_block;
};

RowPlan plan_rows(int vec_per_row)
{
    RowPlan p;
    // two vectors per thread, up to 512 threads per row (measured: the row movers are HBM-bound for any
    // G at H=7168; at H=2048, T=4096 more threads per row shorten the kernel by ~8 %)
    int G = ceil_div(ceil_div(vec_per_row, 2), 32) * 32, U = 2;
    if (G > 512) G = 512;
    if (vec_per_row <= 32) U = 1;
    p.G = G;
    p.U = U;
    p.rows_per_block = G >= kMinBlock ? 1 : kMinBlock / G;
    p.block = G * p.rows_per_block;
    return p;
}

__device__ __forceinline__ void flag_status(int32_t *status, int bits)
{
    if (status) atomicOr(status, bits);
}

// recv[recv_slot[t][k]] = x[t] for the distinct slots of token t.
template <int U>
__global__ void __launch_bounds__(U >= 8 ? 256 : (U == 4 ? 512 : 1024))
dispatch_rows_kernel(const uint4 *__restrict__ x, const int32_t *__restrict__ recv_slot, uint4 *recv,
                     int T, int K, int vec_per_row, int G, long long capacity_rows, int32_t *status)
{
    const int lane = threadIdx.x & 31;
    const int g = threadIdx.x % G;                       // position inside the row group
    const int t = blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
    pdl_trigger();     // a kernel launched behind this one with programmatic serialisation may become resident
    if (t >= T) return;                                   // whole warps leave together (G % 32 == 0)

    // The first row loads do not depend on the slots: they are issued first. When the kernel was launched
    // with programmatic stream serialisation behind the layout (ep_layout_dispatch: x is an input of that
    // call and complete before the layout starts), this is where it waits for the slots to exist; in an
    // ordinary launch the wait returns at once.
    const uint4 *src = x + (size_t)t * vec_per_row;
    uint4 buf[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int v = g + u * G;
        if (v < vec_per_row) buf[u] = ld_stream(src + v);
    }
    pdl_wait();
    int32_t slot = lane < K ? __ldg(recv_slot + (size_t)t * K + lane) : -1;
    if (slot >= capacity_rows) {
        flag_status(status, EP_STATUS_CAPACITY);
        slot = -1;
    }
    // the k's of a token that land on one rank share a slot: keep the lowest k
    const unsigned same = __match_any_sync(kFullMask, slot);
    const unsigned todo = __ballot_sync(kFullMask, slot >= 0 && (same & lanemask_lt()) == 0);

    for (int base = 0; base < vec_per_row; base += G * U) {  // trip count uniform over the warp
        const int v0 = base + g;
        if (base > 0) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * G;
                if (v < vec_per_row) buf[u] = ld_stream(src + v);
            }
        }
        for (unsigned m = todo; m; m &= m - 1) {
            const int32_t row = __shfl_sync(kFullMask, slot, __ffs(m) - 1);
            uint4 *dst = recv + (size_t)row * vec_per_row;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * G;
                if (v < vec_per_row) st_stream(dst + v, buf[u]);
            }
        }
    }
}

// grouped[p] = recv[pair_row[p]] for p < P = *n_pairs.
template <int U>
__global__ void __launch_bounds__(U >= 8 ? 256 : (U == 4 ? 512 : 1024))
group_rows_kernel(const uint4 *__restrict__ recv, long long recv_rows, const int32_t *__restrict__ pair_row,
                  const int32_t *__restrict__ n_pairs, uint4 *grouped, long long capacity_rows,
                  int vec_per_row, int G, int32_t *status)
{
    const int g = threadIdx.x % G;
    const long long p = (long long)blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
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
    for (int v0 = g; v0 < vec_per_row; v0 += G * U) {
        uint4 buf[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) buf[u] = ld_stream(src + v);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) st_stream(dst + v, buf[u]);
        }
    }
}

// dst[dst_slot[i]] = src[src_slot[i]] for i in [0, n): the local grouping written pair by pair, so that
// it can run on any contiguous range of pairs (a token chunk) as soon as that chunk's rows exist.
template <int U>
__global__ void __launch_bounds__(U >= 8 ? 256 : (U == 4 ? 512 : 1024))
permute_rows_kernel(const uint4 *__restrict__ src, long long src_rows, const int32_t *__restrict__ src_slot,
                    uint4 *dst, long long dst_rows, const int32_t *__restrict__ dst_slot, long long n,
                    int vec_per_row, int G, int32_t *status)
{
    const int g = threadIdx.x % G;
    const long long i = (long long)blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
    if (i >= n) return;
    const int32_t s = __ldg(src_slot + i), d = __ldg(dst_slot + i);
    if (s < 0 || d < 0) return;                           // masked pair
    if (s >= src_rows || d >= dst_rows) {
        if (g == 0) flag_status(status, EP_STATUS_CAPACITY);
        return;
    }
    const uint4 *from = src + (size_t)s * vec_per_row;
    uint4 *to = dst + (size_t)d * vec_per_row;
    for (int v0 = g; v0 < vec_per_row; v0 += G * U) {
        uint4 buf[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) buf[u] = ld_stream(from + v);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * G;
            if (v < vec_per_row) st_stream(to + v, buf[u]);
        }
    }
}


}  // namespace

int launch_permute(int hidden, const void *src, int64_t src_rows, const int32_t *src_slot, void *dst,
                   int64_t dst_rows, const int32_t *dst_slot, int64_t n, int32_t *status, cudaStream_t stream)
{
    if (n <= 0) return EP_OK;
    const int vpr = hidden / 8;
    const RowPlan p = plan_rows(vpr);
    const unsigned grid = (unsigned)((n + p.rows_per_block - 1) / p.rows_per_block);
    const uint4 *s4 = static_cast<const uint4 *>(src);
    uint4 *d4 = static_cast<uint4 *>(dst);
    if (p.U == 1)
        permute_rows_kernel<1><<<grid, p.block, 0, stream>>>(s4, src_rows, src_slot, d4, dst_rows, dst_slot, n, vpr, p.G, status);
    else
        permute_rows_kernel<2><<<grid, p.block, 0, stream>>>(s4, src_rows, src_slot, d4, dst_rows, dst_slot, n, vpr, p.G, status);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

int launch_dispatch(const ep_shape_t &s, const void *x, const int32_t *recv_slot, void *recv,
                    int64_t capacity_rows, int32_t *status, cudaStream_t stream, bool behind_layout)
{
    const int T = s.num_tokens, K = s.top_k, vpr = s.hidden / 8;
    const uint4 *xs = static_cast<const uint4 *>(x);
    uint4 *rd = static_cast<uint4 *>(recv);
    const RowPlan p = plan_rows(vpr);
    const int grid = ceil_div(T, p.rows_per_block);
    // behind_layout: the CTAs may become resident (and load their rows) while the layout kernel still runs
    const long long cap = capacity_rows;
    const dim3 g3(grid), b3(p.block);
    cudaError_t e;
    switch (p.U) {
    case 1: e = launch_kernel(behind_layout, dispatch_rows_kernel<1>, g3, b3, 0, stream, xs, recv_slot, rd, T, K, vpr, p.G, cap, status); break;
    case 2: e = launch_kernel(behind_layout, dispatch_rows_kernel<2>, g3, b3, 0, stream, xs, recv_slot, rd, T, K, vpr, p.G, cap, status); break;
    case 4: e = launch_kernel(behind_layout, dispatch_rows_kernel<4>, g3, b3, 0, stream, xs, recv_slot, rd, T, K, vpr, p.G, cap, status); break;
    default: e = launch_kernel(behind_layout, dispatch_rows_kernel<8>, g3, b3, 0, stream, xs, recv_slot, rd, T, K, vpr, p.G, cap, status);
    }
    EP_CUDA_TRY(e);
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
    const RowPlan p = plan_rows(vpr);
    const unsigned grid = (unsigned)((max_pairs + p.rows_per_block - 1) / p.rows_per_block);
    switch (p.U) {
    case 1: group_rows_kernel<1><<<grid, p.block, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, p.G, status); break;
    case 2: group_rows_kernel<2><<<grid, p.block, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, p.G, status); break;
    case 4: group_rows_kernel<4><<<grid, p.block, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, p.G, status); break;
    default: group_rows_kernel<8><<<grid, p.block, 0, stream>>>(rs, recv_rows, pair_row, n_pairs, gd, capacity_rows, vpr, p.G, status);
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
