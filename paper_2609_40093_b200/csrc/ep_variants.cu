// Variants around the hot path, built from the same row-mover pattern (a group of G
// threads per token, 16-byte columns, fp32 fused multiply-add chains in k order):
//   ep_combine_partial         combine with one partial output row per (token, rank)
//   ep_dense_allgather         dense dispatch: every rank receives every token
//   ep_dense_reduce_scatter    dense combine: per-rank buffers ordered by source token,
//                              summed over the ranks
#include "ep_common.cuh"

namespace ep {
namespace {

constexpr int kMinBlock = 128;
constexpr int kChunk = 8;   // rows in flight per column

__device__ __forceinline__ void fma8(float (&acc)[8], float w, const uint4 &r)
{
    acc[0] = __fmaf_rn(w, bf16_lo(r.x), acc[0]);
    acc[1] = __fmaf_rn(w, bf16_hi(r.x), acc[1]);
    acc[2] = __fmaf_rn(w, bf16_lo(r.y), acc[2]);
    acc[3] = __fmaf_rn(w, bf16_hi(r.y), acc[3]);
    acc[4] = __fmaf_rn(w, bf16_lo(r.z), acc[4]);
    acc[5] = __fmaf_rn(w, bf16_hi(r.z), acc[5]);
    acc[6] = __fmaf_rn(w, bf16_lo(r.w), acc[6]);
    acc[7] = __fmaf_rn(w, bf16_hi(r.w), acc[7]);
}

__device__ __forceinline__ uint4 pack8(const float (&acc)[8])
{
    uint4 o;
    o.x = pack_bf16x2(acc[0], acc[1]);
    o.y = pack_bf16x2(acc[2], acc[3]);
    o.z = pack_bf16x2(acc[4], acc[5]);
    o.w = pack_bf16x2(acc[6], acc[7]);
    return o;
}

struct GroupPlan {
    int G, block, rows_per_block;
};

GroupPlan plan_group(int vec_per_row)
{
    GroupPlan p;
    p.G = ceil_div(ceil_div(vec_per_row, ceil_div(vec_per_row, 256)), 32) * 32;   // <= 256 threads, whole columns per thread
    p.rows_per_block = p.G >= kMinBlock ? 1 : kMinBlock / p.G;
    p.block = p.G * p.rows_per_block;
    return p;
}

// Stage 1 of a two-stage combine. For token t the k's are partitioned by a key (the
// receive row in the routed form, the destination rank in the dense form); for
// every part, dst[row(part)] = bf16( fma chain over the part's k in ascending order ).
// Dense form: parts are the ranks 0..R-1, row = r*T + t, empty parts write +0.
__global__ void __launch_bounds__(256, 3)
reduce_to_rows_kernel(const uint4 *__restrict__ out, long long out_rows, const int32_t *__restrict__ pair_slot,
                      const int32_t *__restrict__ recv_slot, const int32_t *__restrict__ topk_idx,
                      const float *__restrict__ weights, uint4 *dst, long long dst_rows, int T, int K, int E, int R,
                      int vec_per_row, int G, int32_t *status)
{
    const int lane = threadIdx.x & 31;
    const int g = threadIdx.x % G;
    const int t = blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
    if (t >= T) return;                                   // whole warps leave together (G % 32 == 0)
    const bool dense = recv_slot == nullptr;

    int32_t my_pair = -1, my_key = -1;
    float my_w = 0.f;
    if (lane < K) {
        my_pair = __ldg(pair_slot + (size_t)t * K + lane);
        my_w = __ldg(weights + (size_t)t * K + lane);
        if (dense) {
            const int e = __ldg(topk_idx + (size_t)t * K + lane);
            my_key = (e >= 0 && e < E) ? e / (E / R) : -1;
        } else {
            my_key = __ldg(recv_slot + (size_t)t * K + lane);
        }
        if (my_pair >= out_rows || (my_key >= 0 && my_pair < 0)) {
            if (status) atomicOr(status, EP_STATUS_CAPACITY);
            my_key = -1;
        }
        if (my_pair < 0) my_key = -1;
    }
    const unsigned same = __match_any_sync(kFullMask, my_key);
    const unsigned firsts = __ballot_sync(kFullMask, my_key >= 0 && (same & lanemask_lt()) == 0);
    const int n_parts = dense ? R : __popc(firsts);

    // part -> (member lanes, destination row); uniform over the warp
    auto part_of = [&](int part, unsigned &todo, unsigned &members, long long &row) {
        if (dense) {
            members = __ballot_sync(kFullMask, my_key == part);
            row = (long long)part * T + t;
        } else {
            const int leader = __ffs(todo) - 1;
            todo &= todo - 1;
            members = __shfl_sync(kFullMask, same, leader);
            row = __shfl_sync(kFullMask, my_key, leader);
        }
        if (row >= dst_rows) {
            if (lane == 0 && status) atomicOr(status, EP_STATUS_CAPACITY);
            return false;
        }
        return true;
    };

    if (K <= kChunk) {
        // all K rows of a column are loaded once (K loads in flight), then every part folds its members
        float wreg[kChunk];
#pragma unroll
        for (int j = 0; j < kChunk; ++j) wreg[j] = __shfl_sync(kFullMask, my_w, j);
        for (int base = 0; base < vec_per_row; base += G) {   // trip count uniform over the warp
            const int v = base + g;
            const bool live = v < vec_per_row;
            uint4 rowv[kChunk];
#pragma unroll
            for (int j = 0; j < kChunk; ++j) {
                const int32_t p = __shfl_sync(kFullMask, my_pair, j);
                const int32_t key = __shfl_sync(kFullMask, my_key, j);
                if (live && key >= 0) rowv[j] = ld_stream(out + (size_t)p * vec_per_row + v);
            }
            unsigned todo = firsts;
            for (int part = 0; part < n_parts; ++part) {
                unsigned members;
                long long row;
                if (!part_of(part, todo, members, row)) continue;
                float acc[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
                for (int j = 0; j < kChunk; ++j)
                    if ((members >> j) & 1u)
                        if (live) fma8(acc, wreg[j], rowv[j]);
                if (live) st_stream(dst + (size_t)row * vec_per_row + v, pack8(acc));
            }
        }
        return;
    }

    unsigned todo = firsts;
    for (int part = 0; part < n_parts; ++part) {
        unsigned members;
        long long row;
        if (!part_of(part, todo, members, row)) continue;
        uint4 *drow = dst + (size_t)row * vec_per_row;
        for (int base = 0; base < vec_per_row; base += G) {   // trip count uniform over the warp
            const int v = base + g;
            const bool live = v < vec_per_row;
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
            unsigned mm = members;
            while (mm) {                                  // the part's k in ascending order, kChunk rows in flight
                uint4 rowv[kChunk];
                int src_lane[kChunk];
#pragma unroll
                for (int j = 0; j < kChunk; ++j) {
                    src_lane[j] = -1;
                    if (mm) {
                        src_lane[j] = __ffs(mm) - 1;
                        mm &= mm - 1;
                        const int32_t p = __shfl_sync(kFullMask, my_pair, src_lane[j]);
                        if (live) rowv[j] = ld_stream(out + (size_t)p * vec_per_row + v);
                    }
                }
#pragma unroll
                for (int j = 0; j < kChunk; ++j)
                    if (src_lane[j] >= 0) {
                        const float w = __shfl_sync(kFullMask, my_w, src_lane[j]);
                        if (live) fma8(acc, w, rowv[j]);
                    }
            }
            if (live) st_stream(drow + v, pack8(acc));
        }
    }
}

// Stage 2: y[t] = bf16( fp32 sum from +0 of the rows the token names ). Routed form: the
// token's distinct receive rows in the order of their first k (slot table with
// duplicates). Dense form (slot == nullptr): rows r*T + t for r = 0..R-1.
__global__ void __launch_bounds__(256, 4)
sum_rows_kernel(const uint4 *__restrict__ src, long long src_rows, const int32_t *__restrict__ slot,
                uint4 *__restrict__ y, int T, int K, int vec_per_row, int G, int32_t *status)
{
    const int lane = threadIdx.x & 31;
    const int g = threadIdx.x % G;
    const int t = blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
    if (t >= T) return;
    long long my_row = -1;
    if (lane < K) {
        my_row = slot ? (long long)__ldg(slot + (size_t)t * K + lane) : (long long)lane * T + t;
        if (my_row >= src_rows) {
            if (status) atomicOr(status, EP_STATUS_CAPACITY);
            my_row = -1;
        }
    }
    const unsigned same = __match_any_sync(kFullMask, my_row);
    const unsigned rows = __ballot_sync(kFullMask, my_row >= 0 && (same & lanemask_lt()) == 0);
    uint4 *dst = y + (size_t)t * vec_per_row;
    for (int base = 0; base < vec_per_row; base += G) {
        const int v = base + g;
        const bool live = v < vec_per_row;
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        unsigned mm = rows;
        while (mm) {
            uint4 rowv[kChunk];
            unsigned have = 0;
#pragma unroll
            for (int j = 0; j < kChunk; ++j)
                if (mm) {
                    const int l = __ffs(mm) - 1;
                    mm &= mm - 1;
                    const long long r = __shfl_sync(kFullMask, my_row, l);
                    if (live) rowv[j] = ld_stream(src + (size_t)r * vec_per_row + v);
                    have |= 1u << j;
                }
#pragma unroll
            for (int j = 0; j < kChunk; ++j)
                if ((have >> j) & 1u)
                    if (live) fma8(acc, 1.0f, rowv[j]);       // 1*v + acc: one rounding, the plain fp32 sum
        }
        if (live) st_stream(dst + v, pack8(acc));
    }
}

// Dense dispatch: gathered[r*T + t] = x[t] for every rank r.
__global__ void __launch_bounds__(512)
dense_allgather_kernel(const uint4 *__restrict__ x, uint4 *gathered, int T, int R, int vec_per_row, int G)
{
    const int g = threadIdx.x % G;
    const int t = blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
    if (t >= T) return;
    const uint4 *src = x + (size_t)t * vec_per_row;
    for (int v0 = g; v0 < vec_per_row; v0 += 2 * G) {
        const int v1 = v0 + G;
        uint4 a = ld_stream(src + v0), b = a;
        if (v1 < vec_per_row) b = ld_stream(src + v1);
        for (int r = 0; r < R; ++r) {
            uint4 *dst = gathered + ((size_t)r * T + t) * vec_per_row;
            st_stream(dst + v0, a);
            if (v1 < vec_per_row) st_stream(dst + v1, b);
        }
    }
}

}  // namespace

// Stage 1 of the routed two-stage combine: partial[recv_slot[t][k]] = bf16(fma chain of the k's sharing that row).
int launch_partial_rows(const ep_shape_t &s, const void *out, int64_t out_rows, const int32_t *pair_slot,
                        const int32_t *recv_slot, const float *weights, void *partial, int64_t partial_rows,
                        int32_t *status, cudaStream_t stream)
{
    const int T = s.num_tokens, vpr = s.hidden / 8;
    const GroupPlan p = plan_group(vpr);
    reduce_to_rows_kernel<<<ceil_div(T, p.rows_per_block), p.block, 0, stream>>>(
        static_cast<const uint4 *>(out), out_rows, pair_slot, recv_slot, nullptr, weights, static_cast<uint4 *>(partial),
        partial_rows, T, s.top_k, s.num_experts, s.num_ranks, vpr, p.G, status);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

// Stage 2 for `n_tokens` tokens starting at the rows the pointers name: y[t] = bf16(sum of the token's
// distinct partial rows in the order of their first k). slot and y point at the first token of the range.
int launch_sum_partial_rows(int hidden, int top_k, const void *partial, int64_t partial_rows, const int32_t *slot,
                            void *y, int n_tokens, int32_t *status, cudaStream_t stream)
{
    if (n_tokens <= 0) return EP_OK;
    const int vpr = hidden / 8;
    const GroupPlan p = plan_group(vpr);
    sum_rows_kernel<<<ceil_div(n_tokens, p.rows_per_block), p.block, 0, stream>>>(
        static_cast<const uint4 *>(partial), partial_rows, slot, static_cast<uint4 *>(y), n_tokens, top_k, vpr, p.G, status);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

}  // namespace ep

extern "C" int ep_combine_partial(const ep_shape_t *shape, const void *out, int64_t out_rows,
                                  const int32_t *pair_slot, const int32_t *recv_slot, const float *topk_weights,
                                  void *partial, int64_t partial_capacity_rows, void *y, int32_t *status,
                                  void *stream_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!out || !pair_slot || !recv_slot || !topk_weights || !partial || !y) return EP_ERR_NULL;
    if (!aligned16(out) || !aligned16(partial) || !aligned16(y) || out_rows < 0 || partial_capacity_rows < 0)
        return EP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    rc = launch_partial_rows(*shape, out, out_rows, pair_slot, recv_slot, topk_weights, partial, partial_capacity_rows,
                             status, stream);
    if (rc != EP_OK) return rc;
    return launch_sum_partial_rows(shape->hidden, shape->top_k, partial, partial_capacity_rows, recv_slot, y,
                                   shape->num_tokens, status, stream);
}

extern "C" int ep_dense_allgather(const ep_shape_t *shape, const void *x, void *gathered, void *stream_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x || !gathered) return EP_ERR_NULL;
    if (!aligned16(x) || !aligned16(gathered)) return EP_ERR_INVALID_ARG;
    const int T = shape->num_tokens, vpr = shape->hidden / 8;
    int G = ceil_div(ceil_div(vpr, 2), 32) * 32;
    if (G > 512) G = 512;
    const int rows_per_block = G >= kMinBlock ? 1 : kMinBlock / G;
    dense_allgather_kernel<<<ceil_div(T, rows_per_block), G * rows_per_block, 0, static_cast<cudaStream_t>(stream_)>>>(
        static_cast<const uint4 *>(x), static_cast<uint4 *>(gathered), T, shape->num_ranks, vpr, G);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

extern "C" int ep_dense_reduce_scatter(const ep_shape_t *shape, const int32_t *topk_idx, const void *out,
                                       int64_t out_rows, const int32_t *pair_slot, const float *topk_weights,
                                       void *dense, void *y, int32_t *status, void *stream_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_ranks > 32) return EP_ERR_INVALID_ARG;     // one lane per rank in the final sum
    if (shape->num_tokens == 0) return EP_OK;
    if (!topk_idx || !out || !pair_slot || !topk_weights || !dense || !y) return EP_ERR_NULL;
    if (!aligned16(out) || !aligned16(dense) || !aligned16(y) || out_rows < 0) return EP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int T = shape->num_tokens, K = shape->top_k, R = shape->num_ranks, vpr = shape->hidden / 8;
    const GroupPlan p = plan_group(vpr);
    const int grid = ceil_div(T, p.rows_per_block);
    const long long dense_rows = (long long)R * T;
    reduce_to_rows_kernel<<<grid, p.block, 0, stream>>>(static_cast<const uint4 *>(out), out_rows, pair_slot, nullptr,
                                                        topk_idx, topk_weights, static_cast<uint4 *>(dense), dense_rows,
                                                        T, K, shape->num_experts, R, vpr, p.G, status);
    sum_rows_kernel<<<grid, p.block, 0, stream>>>(static_cast<const uint4 *>(dense), dense_rows, nullptr,
                                                  static_cast<uint4 *>(y), T, R, vpr, p.G, status);
    EP_LAUNCH_CHECK(2);
    return EP_OK;
}
