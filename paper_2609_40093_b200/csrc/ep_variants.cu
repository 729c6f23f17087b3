// Variants around the hot path:
//   ep_combine_partial         combine with one partial output row per (token, rank)
//   ep_dense_allgather         dense dispatch: every rank receives every token
//   ep_dense_reduce_scatter    dense combine: per-rank buffers ordered by source token,
//                              summed over the ranks
// The two-stage combines run on the combine kernel's segmented and distinct-row modes
// (ep_combine.cu); this file holds the dense all-gather's row mover and the entry points.
#include "ep_common.cuh"

namespace ep {
namespace {

constexpr int kMinBlock = 128;

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
    rc = launch_partial_rows(*shape, out, out_rows, pair_slot, recv_slot, 0, topk_weights, partial,
                             partial_capacity_rows, status, stream);
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
    if ((int64_t)shape->num_ranks * shape->num_tokens >= (int64_t(1) << 31)) return EP_ERR_INVALID_ARG;
    if (shape->num_tokens == 0) return EP_OK;
    if (!topk_idx || !out || !pair_slot || !topk_weights || !dense || !y) return EP_ERR_NULL;
    if (!aligned16(out) || !aligned16(dense) || !aligned16(y) || out_rows < 0) return EP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int T = shape->num_tokens, R = shape->num_ranks;
    const long long dense_rows = (long long)R * T;
    rc = launch_partial_rows(*shape, out, out_rows, pair_slot, topk_idx, 1, topk_weights, dense, dense_rows, status, stream);
    if (rc != EP_OK) return rc;
    return launch_sum_partial_rows(shape->hidden, R, dense, dense_rows, nullptr, y, T, status, stream);
}
