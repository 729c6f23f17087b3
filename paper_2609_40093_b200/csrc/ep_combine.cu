// ep_combine and the reductions of the two-stage combines: one kernel, three modes.
//
//   plain      y[t] = bf16( sum_k w[t][k] * out[slot[t][k]] ), fp32 fused multiply-add chain from
//              +0 in ascending k, one rounding to bf16 at the end (ep_combine);
//   segmented  stage 1 of a two-stage combine: the token's k are partitioned by a key (the receive
//              row in the routed form, the expert's rank in the dense form); each part's chain
//              (ascending k, from +0) is rounded to bf16 and stored to the part's row;
//   distinct   stage 2: y[t] = bf16( fp32 sum from +0 of the distinct rows the token names, in the
//              order of their first k ), unit weights (1*v + acc is the plain fp32 add).
//
// A group of G threads (32, 64 or 128) owns one token; each thread owns 16-byte columns (8 bf16).
// For a column it first issues the loads of up to kChunk rows (they are independent: this is the
// memory-level parallelism), then folds them into the eight accumulators strictly in order. Slots
// and weights sit one per lane and travel by warp shuffle. For K <= 8 the rows of a column are
// requested in two halves and the next column's halves are requested between the two folds, so that
// loads stay in flight during the arithmetic (measured -2 us of 166 at T=8192, H=7168, K=8). Small
// CTAs (128 threads, at most 64 registers, eight resident per SM) measured 5 % faster alone than
// 448-thread groups with two columns per thread (165 vs 175 us at T=8192, H=7168, K=8).
//
// Segmented mode sorts the token's valid entries by (part, k) once per warp (K <= 32 entries, by
// shuffles), so that the column loop is the plain chain with two warp-uniform bit masks: "a part
// starts here" and "a part ends here: round, store, clear". Every row is still loaded once and every
// product is one fused multiply-add: the work per column is that of the plain mode plus the stores.
#include "ep_common.cuh"

namespace ep {
namespace {

constexpr int kBlock = 128;
constexpr int kChunk = 8;   // rows in flight per column
constexpr int kParts = 2;   // K <= 8: groups the rows of a column are requested in (4 and 8 measured the same)

enum { kPlain = 0, kDistinct = 1, kSegmented = 2 };

struct CombineArgs {
    const uint4 *out;           // source rows
    long long out_rows;
    const int32_t *slot;        // plain: slot table; distinct: slot table, or NULL for rows lane*T + t; segmented: pair_slot
    const int32_t *key;         // segmented: recv_slot (routed) or topk_idx (dense)
    const float *weights;       // plain, segmented
    uint4 *y;                   // plain, distinct: [T] rows; segmented: destination rows
    long long y_rows;           // segmented: capacity of the destination
    int T, K, vec_per_row;
    int E, R;                   // segmented, dense form: expert -> rank; parts are the ranks 0..R-1
    int dense;
    int32_t *status;
};

__device__ __forceinline__ void fma_row(float (&acc)[8], float w, const uint4 &r)
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

__device__ __forceinline__ uint4 pack_row(const float (&acc)[8])
{
    uint4 o;
    o.x = pack_bf16x2(acc[0], acc[1]);
    o.y = pack_bf16x2(acc[2], acc[3]);
    o.z = pack_bf16x2(acc[4], acc[5]);
    o.w = pack_bf16x2(acc[6], acc[7]);
    return o;
}

template <int G, int MODE>
__global__ void __launch_bounds__(kBlock)
combine_rows_kernel(const CombineArgs a)
{
    const int lane = threadIdx.x & 31;
    const int g = threadIdx.x % G;
    const int t = blockIdx.x * (kBlock / G) + threadIdx.x / G;
    // launched with programmatic stream serialisation: the CTAs may be resident before the previous
    // kernel of the stream has finished; nothing is read or written before this returns
    pdl_wait();
    if (t >= a.T) return;                                 // whole warps leave together (G >= 32)
    const int K = a.K, vec_per_row = a.vec_per_row;

    // ---- this token's entries, one per lane: source row, weight, (segmented) destination row
    int32_t my_slot = -1, my_dst = -1;
    float my_w = 0.f;
    unsigned ends = 0u;          // segmented: entries after which a part is rounded and stored
    unsigned absent = 0u;        // segmented, dense form: ranks that hold nothing of this token (zero rows)
    int n = K;                   // entries the column loop walks
    if (MODE == kPlain) {
        if (lane < K) {
            my_slot = __ldg(a.slot + (size_t)t * K + lane);
            my_w = __ldg(a.weights + (size_t)t * K + lane);
        }
    } else if (MODE == kDistinct) {
        if (lane < K) my_slot = a.slot ? __ldg(a.slot + (size_t)t * K + lane) : lane * a.T + t;
        my_w = 1.0f;
    } else {
        int32_t pair = -1, key = -1;
        float w = 0.f;
        if (lane < K) {
            pair = __ldg(a.slot + (size_t)t * K + lane);
            w = __ldg(a.weights + (size_t)t * K + lane);
            if (a.dense) {
                const int e = __ldg(a.key + (size_t)t * K + lane);
                key = (e >= 0 && e < a.E) ? e / (a.E / a.R) : -1;
            } else {
                key = __ldg(a.key + (size_t)t * K + lane);
            }
            if (pair >= a.out_rows || (key >= 0 && pair < 0)) {
                if (a.status) atomicOr(a.status, EP_STATUS_CAPACITY);
                key = -1;
            }
            if (pair < 0) key = -1;
        }
        // order of the entries: by part, then k. Routed form: parts in the order of their first k;
        // dense form: parts are the ranks in ascending order.
        const unsigned same = __match_any_sync(kFullMask, key);
        const bool valid = key >= 0;
        const int part = a.dense ? key : __ffs(same) - 1;
        const int composite = valid ? (part << 5 | lane) : 0x7fffffff;
        int pos = 0;
        for (int j = 0; j < K; ++j) pos += __shfl_sync(kFullMask, composite, j) < composite;
        const unsigned valid_mask = __ballot_sync(kFullMask, valid);
        n = __popc(valid_mask);
        int src = 0;                                      // the entry that belongs at position `lane`
        for (int j = 0; j < K; ++j) {
            const int p = __shfl_sync(kFullMask, pos, j);
            if (((valid_mask >> j) & 1u) && p == lane) src = j;
        }
        my_slot = __shfl_sync(kFullMask, pair, src);
        my_w = __shfl_sync(kFullMask, w, src);
        const int32_t skey = __shfl_sync(kFullMask, key, src);
        const int32_t next_key = __shfl_down_sync(kFullMask, skey, 1);
        const bool in = lane < n;
        if (!in) my_slot = -1;
        my_dst = a.dense ? skey * a.T + t : skey;
        const bool last = in && (lane == n - 1 || next_key != skey);
        const bool fits = my_dst < a.y_rows;
        if (last && !fits && a.status) atomicOr(a.status, EP_STATUS_CAPACITY);
        ends = __ballot_sync(kFullMask, last);
        if (!fits) my_dst = -1;                           // a part whose row does not fit is computed and dropped
        if (a.dense) {
            unsigned present = 0u;
            for (int r = 0; r < a.R; ++r)
                if (__ballot_sync(kFullMask, valid && key == r)) present |= 1u << r;
            absent = ~present & (a.R >= 32 ? 0xffffffffu : ((1u << a.R) - 1u));
        }
    }
    if (MODE != kSegmented && lane < K && my_slot >= a.out_rows) {
        if (a.status) atomicOr(a.status, EP_STATUS_CAPACITY);
        my_slot = -1;
    }
    if (MODE == kDistinct) {                              // a row named twice counts once: keep its first k
        const unsigned same = __match_any_sync(kFullMask, my_slot);
        if ((same & lanemask_lt()) != 0) my_slot = -1;
    }
    uint4 *dst = a.y + (size_t)t * vec_per_row;           // plain, distinct
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);

    if (K <= kChunk) {
        // K <= 8: the rows of a column are requested in kParts groups, and each group of the next column
        // is requested right after the same group of this column has been folded, so that most loads
        // stay in flight during the arithmetic. The chain order is unchanged.
        constexpr int kPer = kChunk / kParts;
        const unsigned valid = __ballot_sync(kFullMask, my_slot >= 0);
        uint4 row[kParts][kPer];
        int v = g;
        bool live = v < vec_per_row;
#pragma unroll
        for (int p = 0; p < kParts; ++p)
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int k = p * kPer + j;
                const int32_t s = __shfl_sync(kFullMask, my_slot, k);
                if (live && ((valid >> k) & 1u)) row[p][j] = ld_stream(a.out + (size_t)s * vec_per_row + v);
            }
        for (int base = 0; base < vec_per_row; base += G) {   // trip count uniform over the warp
            const int vn = v + G;
            const bool live_n = vn < vec_per_row;
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
            for (int p = 0; p < kParts; ++p) {
#pragma unroll
                for (int j = 0; j < kPer; ++j) {
                    const int k = p * kPer + j;
                    const float w = __shfl_sync(kFullMask, my_w, k);
                    if (live && ((valid >> k) & 1u)) fma_row(acc, w, row[p][j]);
                    if (MODE == kSegmented && ((ends >> k) & 1u)) {     // warp-uniform: a part ends here
                        const int32_t d = __shfl_sync(kFullMask, my_dst, k);
                        if (live && d >= 0) st_stream(a.y + (size_t)d * vec_per_row + v, pack_row(acc));
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
                    }
                }
#pragma unroll
                for (int j = 0; j < kPer; ++j) {             // the same group of the next column
                    const int k = p * kPer + j;
                    const int32_t s = __shfl_sync(kFullMask, my_slot, k);
                    if (live_n && ((valid >> k) & 1u)) row[p][j] = ld_stream(a.out + (size_t)s * vec_per_row + vn);
                }
            }
            if (MODE == kSegmented) {
                if (live)
                    for (unsigned m = absent; m; m &= m - 1)     // dense form: ranks without a pick hold +0
                        st_stream(a.y + ((size_t)(__ffs(m) - 1) * a.T + t) * vec_per_row + v, zero);
            } else if (live) {
                st_stream(dst + v, pack_row(acc));
            }
            v = vn;
            live = live_n;
        }
        return;
    }
    for (int base = 0; base < vec_per_row; base += G) {   // trip count uniform over the warp
        const int v = base + g;
        const bool live = v < vec_per_row;
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        for (int k0 = 0; k0 < n; k0 += kChunk) {
            uint4 row[kChunk];
            int32_t s[kChunk];
#pragma unroll
            for (int j = 0; j < kChunk; ++j) {
                s[j] = __shfl_sync(kFullMask, my_slot, (k0 + j) & 31);
                if (k0 + j >= n) s[j] = -1;
                if (live && s[j] >= 0) row[j] = ld_stream(a.out + (size_t)s[j] * vec_per_row + v);
            }
#pragma unroll
            for (int j = 0; j < kChunk; ++j) {
                const float w = __shfl_sync(kFullMask, my_w, (k0 + j) & 31);
                if (live && s[j] >= 0) fma_row(acc, w, row[j]);
                if (MODE == kSegmented && k0 + j < n && ((ends >> (k0 + j)) & 1u)) {
                    const int32_t d = __shfl_sync(kFullMask, my_dst, k0 + j);
                    if (live && d >= 0) st_stream(a.y + (size_t)d * vec_per_row + v, pack_row(acc));
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
                }
            }
        }
        if (MODE == kSegmented) {
            if (live)
                for (unsigned m = absent; m; m &= m - 1)
                    st_stream(a.y + ((size_t)(__ffs(m) - 1) * a.T + t) * vec_per_row + v, zero);
        } else if (live) {
            st_stream(dst + v, pack_row(acc));
        }
    }
}

template <int MODE>
int launch_mode(const CombineArgs &a, cudaStream_t stream)
{
    const int vpr = a.vec_per_row, T = a.T;
    const int G = vpr <= 64 ? 32 : (vpr <= 256 ? 64 : 128);
    cudaError_t e;
    if (G == 32)
        e = launch_pdl(combine_rows_kernel<32, MODE>, dim3(ceil_div(T, kBlock / 32)), dim3(kBlock), 0, stream, a);
    else if (G == 64)
        e = launch_pdl(combine_rows_kernel<64, MODE>, dim3(ceil_div(T, kBlock / 64)), dim3(kBlock), 0, stream, a);
    else
        e = launch_pdl(combine_rows_kernel<128, MODE>, dim3(T), dim3(kBlock), 0, stream, a);
    EP_CUDA_TRY(e);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

}  // namespace

int launch_combine(const ep_shape_t &s, const void *out, int64_t out_rows, const int32_t *slot,
                   const float *weights, void *y, int32_t *status, cudaStream_t stream)
{
    CombineArgs a = {};
    a.out = static_cast<const uint4 *>(out);
    a.out_rows = out_rows;
    a.slot = slot;
    a.weights = weights;
    a.y = static_cast<uint4 *>(y);
    a.T = s.num_tokens; a.K = s.top_k; a.vec_per_row = s.hidden / 8;
    a.status = status;
    return launch_mode<kPlain>(a, stream);
}

// Stage 1 of a two-stage combine. Routed form (key = recv_slot): partial[recv_slot[t][k]] = bf16( chain over
// the k that share the row ). Dense form (key = topk_idx, dense != 0): dst[r*T + t] for every rank r, +0 where
// the token has no expert on r.
int launch_partial_rows(const ep_shape_t &s, const void *out, int64_t out_rows, const int32_t *pair_slot,
                        const int32_t *key, int dense, const float *weights, void *partial, int64_t partial_rows,
                        int32_t *status, cudaStream_t stream)
{
    CombineArgs a = {};
    a.out = static_cast<const uint4 *>(out);
    a.out_rows = out_rows;
    a.slot = pair_slot;
    a.key = key;
    a.weights = weights;
    a.y = static_cast<uint4 *>(partial);
    a.y_rows = partial_rows;
    a.T = s.num_tokens; a.K = s.top_k; a.vec_per_row = s.hidden / 8;
    a.E = s.num_experts; a.R = s.num_ranks;
    a.dense = dense;
    a.status = status;
    return launch_mode<kSegmented>(a, stream);
}

// Stage 2 for `n_tokens` tokens starting at the rows the pointers name: y[t] = bf16( sum of the token's distinct
// rows in the order of their first k ). slot == NULL: the dense form, rows r*T + t for r = 0..top_k-1, with
// `partial` pointing at row 0 of the dense buffer and T = n_tokens.
int launch_sum_partial_rows(int hidden, int top_k, const void *partial, int64_t partial_rows, const int32_t *slot,
                            void *y, int n_tokens, int32_t *status, cudaStream_t stream)
{
    if (n_tokens <= 0) return EP_OK;
    CombineArgs a = {};
    a.out = static_cast<const uint4 *>(partial);
    a.out_rows = partial_rows;
    a.slot = slot;
    a.y = static_cast<uint4 *>(y);
    a.T = n_tokens; a.K = top_k; a.vec_per_row = hidden / 8;
    a.status = status;
    return launch_mode<kDistinct>(a, stream);
}

}  // namespace ep

extern "C" int ep_combine(const ep_shape_t *shape, const void *out, int64_t out_rows, const int32_t *slot,
                          const float *topk_weights, void *y, int32_t *status, void *stream)
{
    int rc = ep::check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!out || !slot || !topk_weights || !y) return EP_ERR_NULL;
    if (!ep::aligned16(out) || !ep::aligned16(y) || out_rows < 0) return EP_ERR_INVALID_ARG;
    return ep::launch_combine(*shape, out, out_rows, slot, topk_weights, y, status, static_cast<cudaStream_t>(stream));
}
