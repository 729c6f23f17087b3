// ep_layout_dispatch: layout and dispatch of a small batch in one launch.
//
// Decode-size batches are bound by launch and memory latency, not by bytes. Up to
// 1024 tokens the whole routing table fits in shared memory, so every CTA computes
// the complete layout for itself (no exchange between CTAs, no second launch),
// keeps what concerns its own tokens, writes those tokens' entries of the layout
// arrays, and copies their rows to the destination ranks. The loads of the rows do
// not depend on the layout and are issued before it is computed. CTA 0 also writes
// the small arrays (counts, offsets, per-source segments, status).
//
// Per CTA: own tokens [t0, t0 + tpc), tpc a power of two <= 32, so they lie inside
// one 32-token group g0.
//   1. stage all ids (T*K) in shared memory, odd row stride;
//   2. expert histogram over all pairs and over the pairs of tokens < t0 (shared
//      memory atomics: only sums are used, order does not matter); per 32-token
//      group and rank one ballot of "token hits rank", kept for all groups;
//   3. rank totals and the hits before group g0 from the ballots; one exclusive
//      scan over [experts | ranks];
//   4. warp 0 replays the own tokens in (t,k) order: receive rows from ballots,
//      pair slots from warp matches with running counters that start at
//      expert_offsets[e] + (pairs of e before t0);
//   5. all warps copy the own rows to their distinct destinations.
#include <atomic>
#include <mutex>

#include "ep_common.cuh"
#include "ep_layout_common.cuh"

namespace ep {
namespace {

constexpr int kFusedMaxTokens = 1024;
constexpr int kFusedThreads = 256;
constexpr size_t kFusedMaxSmem = 96 * 1024;
constexpr int kPrefetch = 4;            // 16-byte vectors per thread loaded before the layout is computed

struct FusedArgs {
    const int32_t *idx;
    const uint4 *x;
    uint4 *recv;
    long long capacity_rows;
    ep_layout_t out;
    int T, K, Kp, E, R, Tr;
    uint32_t mul_El, mul_K;
    int tpc;            // tokens per CTA
    int n_groups;       // ceil(T / 32)
    int vec_per_row;
    int wpr;            // warps per row in the copy phase
};

struct FusedPlan {
    bool ok;
    int tpc, n_ctas, wpr;
    size_t smem;
};

inline size_t fused_smem_ints(int n_groups, int Kp, int E, int R)
{
    // ids_all | bal_all | tot[E+R+2] | before_e[E] | grp_before[R] | rows_own[32][Kp] | scan[32]
    return (size_t)n_groups * 32 * Kp + (size_t)n_groups * R + (E + R + 2) + E + R + 32 * (size_t)Kp + 32;
}

FusedPlan plan_fused(const ep_shape_t &s)
{
    FusedPlan p;
    const int T = s.num_tokens, Kp = s.top_k | 1;
    const int n_groups = ceil_div(T > 0 ? T : 1, 32);
    p.smem = sizeof(int32_t) * fused_smem_ints(n_groups, Kp, s.num_experts, s.num_ranks);
    p.ok = T >= 1 && T <= kFusedMaxTokens && p.smem <= kFusedMaxSmem;
    // about 4 KB of input rows per CTA, at most 256 CTAs (every CTA repeats the layout's counting)
    const size_t row_bytes = (size_t)s.hidden * 2;
    int tpc = 1;
    while (tpc < 32 && (size_t)(2 * tpc) * row_bytes <= 4096) tpc *= 2;
    while (tpc < 32 && ceil_div(T, tpc) > 256) tpc *= 2;
    p.tpc = tpc;
    p.n_ctas = ceil_div(T > 0 ? T : 1, tpc);
    const int warps = kFusedThreads / 32;
    p.wpr = tpc >= warps ? 1 : warps / tpc;
    return p;
}

__global__ void __launch_bounds__(kFusedThreads) layout_dispatch_small_kernel(FusedArgs a)
{
    pdl_trigger();                                       // the next kernel of the stream may become resident
    extern __shared__ int32_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kFusedThreads / 32;
    const int nb = a.E + a.R;
    int32_t *ids_all = smem;                                             // [n_groups*32][Kp]
    unsigned *bal_all = reinterpret_cast<unsigned *>(ids_all + a.n_groups * 32 * a.Kp);   // [n_groups][R]
    int32_t *tot = reinterpret_cast<int32_t *>(bal_all + a.n_groups * a.R);               // [E+R+2]
    int32_t *before_e = tot + nb + 2;                                    // [E] pairs of expert e among tokens < t0
    int32_t *grp_before = before_e + a.E;                                // [R] hits of rank r in groups < g0
    int32_t *rows_own = grp_before + a.R;                                // [32][Kp] receive rows of group g0's pairs
    int32_t *sh = rows_own + 32 * a.Kp;                                  // [32]
    const int t0 = blockIdx.x * a.tpc, t_end = min(a.T, t0 + a.tpc), g0 = t0 >> 5;
    const unsigned lt = lanemask_lt();

    // ---- the first vectors of the own rows: independent of the layout, requested now
    const int rows_per_pass = nwarps / a.wpr;            // rows copied at once
    const int sub = warp % a.wpr;                         // this warp's share of a row
    const int stride = a.wpr * 32;
    uint4 pre[kPrefetch];
    {
        const int t = t0 + warp / a.wpr;
#pragma unroll
        for (int u = 0; u < kPrefetch; ++u) {
            const int v = sub * 32 + lane + u * stride;
            if (t < t_end && v < a.vec_per_row) pre[u] = ld_stream(a.x + (size_t)t * a.vec_per_row + v);
        }
    }

    // ---- 1. all ids into shared memory; histograms zeroed
    const int n_pad = a.n_groups * 32 * a.K, n_items = a.T * a.K;
    for (int base = tid; base < n_pad; base += 8 * kFusedThreads) {
        int32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + u * kFusedThreads;
            v[u] = i < n_items ? __ldg(a.idx + i) : -1;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + u * kFusedThreads;
            if (i < n_pad) {
                const int tok = sdiv(i, a.mul_K);
                ids_all[tok * a.Kp + (i - tok * a.K)] = v[u];
            }
        }
    }
    for (int b = tid; b < nb + 2; b += kFusedThreads) tot[b] = 0;
    for (int e = tid; e < a.E; e += kFusedThreads) before_e[e] = 0;
    __syncthreads();

    // ---- 2. expert counts (all pairs; pairs of earlier tokens) and one ballot per (group, rank)
    for (int i = tid; i < n_items; i += kFusedThreads) {
        const int tok = sdiv(i, a.mul_K);
        const int e = ids_all[tok * a.Kp + (i - tok * a.K)];
        if (e >= 0 && e < a.E) {
            atomicAdd(tot + e, 1);
            if (tok < t0) atomicAdd(before_e + e, 1);
        }
    }
    int bad = 0;
    for (int g = warp; g < a.n_groups; g += nwarps) {
        unsigned long long mask = 0ull;
        const int32_t *row = ids_all + (g * 32 + lane) * a.Kp;
        for (int k = 0; k < a.K; ++k) {
            const int e = row[k];
            if (e >= 0 && e < a.E) mask |= 1ull << sdiv(e, a.mul_El);
            else if (e != -1) ++bad;
        }
        for (int r = 0; r < a.R; ++r) {
            const unsigned b = __ballot_sync(kFullMask, (mask >> r) & 1ull);
            if (lane == (r & 31)) bal_all[g * a.R + r] = b;
        }
    }
    if (bad) atomicAdd(tot + nb + 1, bad);               // kept apart from the scanned bins
    __syncthreads();

    // ---- 3. rank totals, hits before the own group; scan over [experts | ranks]
    for (int r = tid; r < a.R; r += kFusedThreads) {
        int32_t total = 0, before = 0;
        for (int g = 0; g < a.n_groups; ++g) {
            const int c = __popc(bal_all[g * a.R + r]);
            total += c;
            if (g < g0) before += c;
        }
        tot[a.E + r] = total;
        grp_before[r] = before;
    }
    __syncthreads();
    const bool first_cta = blockIdx.x == 0;
    if (first_cta) {
        for (int e = tid; e < a.E; e += kFusedThreads) a.out.expert_counts[e] = tot[e];
        for (int r = tid; r < a.R; r += kFusedThreads) a.out.rank_rows[r] = tot[a.E + r];
    }
    __syncthreads();
    block_exclusive_scan_smem(tot, nb, sh);              // tot[e] = expert offset, tot[E+r] - tot[E] = rank row offset
    const int32_t n_pairs = tot[a.E];
    if (first_cta) {
        for (int e = tid; e <= a.E; e += kFusedThreads) a.out.expert_offsets[e] = tot[e];
        for (int r = tid; r <= a.R; r += kFusedThreads) a.out.rank_row_offsets[r] = tot[a.E + r] - n_pairs;
        // first receive row of source rank s inside rank r: hits of r among tokens < s*Tr
        for (int j = tid; j < a.R * (a.R + 1); j += kFusedThreads) {
            const int r = j / (a.R + 1), s = j - r * (a.R + 1);
            const int tb = s * a.Tr, gb = tb >> 5;
            int32_t c = tot[a.E + r] - n_pairs;
            for (int g = 0; g < gb; ++g) c += __popc(bal_all[g * a.R + r]);
            if (gb < a.n_groups) c += __popc(bal_all[gb * a.R + r] & ((1u << (tb & 31)) - 1u));
            a.out.src_row_offsets[j] = c;
        }
        if (tid == 0) {
            const int32_t n_recv = tot[nb] - n_pairs;
            *a.out.status = (tot[nb + 1] ? EP_STATUS_BAD_INDEX : 0) | (n_recv > a.capacity_rows ? EP_STATUS_CAPACITY : 0);
        }
    }

    // ---- 4. warp 0 replays the own tokens (lanes = the 32 tokens of group g0)
    if (warp == 0) {
        const int t = g0 * 32 + lane;
        const bool mine = t >= t0 && t < t_end;
        const int32_t *row_ids = ids_all + t * a.Kp;
        for (int k = 0; k < a.K; ++k) {
            const int e = row_ids[k];
            int32_t row = -1;
            if (e >= 0 && e < a.E) {
                const int r = sdiv(e, a.mul_El);
                row = tot[a.E + r] - n_pairs + grp_before[r] + __popc(bal_all[g0 * a.R + r] & lt);
            }
            rows_own[lane * a.Kp + k] = row;
        }
        for (int r = 0; r < a.R; ++r)                     // receive row -> token: one coalesced store per rank
            if (mine && ((bal_all[g0 * a.R + r] >> lane) & 1u))
                a.out.recv_token[tot[a.E + r] - n_pairs + grp_before[r] + __popc(bal_all[g0 * a.R + r] & lt)] = t;
        __syncwarp();
        const int first_pair = (t0 & 31) * a.K, own_pairs = (t_end - t0) * a.K;
        int32_t *pair_slot = a.out.pair_slot + (size_t)t0 * a.K, *recv_slot = a.out.recv_slot + (size_t)t0 * a.K;
        for (int j = 0; j < own_pairs; j += 32) {
            const int i = j + lane;                      // pair of the own tile, (t,k) order
            const bool act = i < own_pairs;
            const int ig = first_pair + i;               // the same pair inside group g0
            const int tok = sdiv(ig, a.mul_K);
            const int pos = tok * a.Kp + (ig - tok * a.K);
            int e = act ? ids_all[g0 * 32 * a.Kp + pos] : -1;
            if (e >= a.E) e = -2;
            const unsigned m = __match_any_sync(kFullMask, e >= 0 ? e : a.E + lane);
            const int leader = __ffs(m) - 1;
            int32_t first = 0;
            if (e >= 0 && lane == leader) first = tot[e] + atomicAdd(before_e + e, __popc(m));
            first = __shfl_sync(kFullMask, first, leader);
            if (e >= 0) {
                const int32_t p = first + __popc(m & lt);
                const int32_t row = rows_own[pos];
                pair_slot[i] = p;
                recv_slot[i] = row;
                a.out.pair_token[p] = g0 * 32 + tok;
                a.out.pair_row[p] = row;
            } else if (act) {
                pair_slot[i] = -1;
                recv_slot[i] = -1;
            }
            __syncwarp();
        }
    }
    __syncthreads();

    // ---- 5. copy the own rows to their distinct destination rows
    for (int j0 = 0; j0 < a.tpc; j0 += rows_per_pass) {
        const int t = t0 + j0 + warp / a.wpr;
        if (t >= t_end) continue;                         // whole warps skip together
        int32_t slot = lane < a.K ? rows_own[(t & 31) * a.Kp + lane] : -1;
        if (slot >= a.capacity_rows) slot = -1;           // reported by CTA 0 through the row total
        const unsigned same = __match_any_sync(kFullMask, slot);
        const unsigned todo = __ballot_sync(kFullMask, slot >= 0 && (same & lt) == 0);
        const uint4 *src = a.x + (size_t)t * a.vec_per_row;
        for (int base = 0; base < a.vec_per_row; base += stride * kPrefetch) {
            uint4 buf[kPrefetch];
#pragma unroll
            for (int u = 0; u < kPrefetch; ++u) {
                const int v = base + sub * 32 + lane + u * stride;
                if (j0 == 0 && base == 0) buf[u] = pre[u];
                else if (v < a.vec_per_row) buf[u] = ld_stream(src + v);
            }
            for (unsigned mm = todo; mm; mm &= mm - 1) {
                const int32_t row = __shfl_sync(kFullMask, slot, __ffs(mm) - 1);
                uint4 *dst = a.recv + (size_t)row * a.vec_per_row;
#pragma unroll
                for (int u = 0; u < kPrefetch; ++u) {
                    const int v = base + sub * 32 + lane + u * stride;
                    if (v < a.vec_per_row) st_stream(dst + v, buf[u]);
                }
            }
        }
    }
}

}  // namespace
}  // namespace ep

extern "C" int ep_layout_dispatch(const ep_shape_t *shape, const int32_t *topk_idx, const void *x,
                                  const ep_layout_t *out, void *workspace, size_t workspace_bytes, void *recv,
                                  int64_t recv_capacity_rows, void *stream_, void *stream_pairs_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    const FusedPlan plan = plan_fused(*shape);
    if (!plan.ok || (out && topk_idx && layout_is_lean(*shape, topk_idx, *out, workspace ? workspace_bytes : 0))) {
        // larger batches, and every batch the lean layout kernels cover (one small launch of theirs and a dependent
        // dispatch beat the one-launch form: 4.2 against 7.0 us per call at 64 tokens, 8.9 against 13.9 at 1024):
        // the layout, then the dispatch kernel launched with programmatic stream serialisation,
        // so that its CTAs load their rows of x (an input of this call, complete before the layout starts)
        // while the layout still runs, and wait for the slots on the device
        cudaStream_t stream = static_cast<cudaStream_t>(stream_), side = static_cast<cudaStream_t>(stream_pairs_);
        const bool split = stream_pairs_ != nullptr && shape->num_tokens > kFusedMaxTokens;   // small batches gain nothing from it
        cudaEvent_t *ev = nullptr;
        std::unique_lock<std::mutex> hold;
        if (split) {
            // dispatch needs the receive-row half only: the pair half runs on the second stream beside it
            const size_t need = ep_layout_workspace_bytes(shape);
            const size_t half = (need + 255) & ~size_t(255);
            if (!workspace) return EP_ERR_NULL;
            if (workspace_bytes < half + need) return EP_ERR_CAPACITY;
            rc = order_events(&ev, 2, hold);
            if (rc != EP_OK) return rc;
            EP_CUDA_TRY(cudaEventRecord(ev[0], stream));                    // everything queued so far, x and topk_idx included
            EP_CUDA_TRY(cudaStreamWaitEvent(side, ev[0], 0));
            rc = ep_layout_ranks(shape, topk_idx, out, workspace, need, stream_);
            if (rc != EP_OK) return rc;
            rc = ep_layout_pairs(shape, topk_idx, out, static_cast<char *>(workspace) + half, need, stream_pairs_);
            if (rc != EP_OK) return rc;
            EP_CUDA_TRY(cudaEventRecord(ev[1], side));
        } else {
            rc = ep_layout(shape, topk_idx, out, workspace, workspace_bytes, stream_);
            if (rc != EP_OK) return rc;
        }
        if (shape->num_tokens == 0) return EP_OK;
        if (!x || !recv) return EP_ERR_NULL;
        if (!aligned16(x) || !aligned16(recv) || recv_capacity_rows < 0) return EP_ERR_INVALID_ARG;
        rc = launch_dispatch(*shape, x, out->recv_slot, recv, recv_capacity_rows, out->status, stream, true);
        if (rc != EP_OK) return rc;
        if (split) EP_CUDA_TRY(cudaStreamWaitEvent(stream, ev[1], 0));      // the pair half is part of this call's result
        return EP_OK;
    }
    if (!out || !topk_idx || !x || !recv) return EP_ERR_NULL;
    if (!out->expert_counts || !out->expert_offsets || !out->rank_rows || !out->rank_row_offsets ||
        !out->src_row_offsets || !out->recv_slot || !out->pair_slot || !out->recv_token || !out->pair_row ||
        !out->pair_token || !out->status)
        return EP_ERR_NULL;
    if (!aligned16(x) || !aligned16(recv) || recv_capacity_rows < 0) return EP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    static std::atomic<bool> attr_done[64] = {};          // per device: dynamic shared memory limit raised
    int dev = 0;
    EP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return EP_ERR_INVALID_ARG;
    if (!attr_done[dev].load(std::memory_order_acquire)) {
        EP_CUDA_TRY(cudaFuncSetAttribute(layout_dispatch_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kFusedMaxSmem));
        attr_done[dev].store(true, std::memory_order_release);
    }
    FusedArgs a;
    a.idx = topk_idx;
    a.x = static_cast<const uint4 *>(x);
    a.recv = static_cast<uint4 *>(recv);
    a.capacity_rows = recv_capacity_rows;
    a.out = *out;
    a.T = shape->num_tokens; a.K = shape->top_k; a.Kp = shape->top_k | 1; a.E = shape->num_experts; a.R = shape->num_ranks;
    a.Tr = a.T / a.R;
    a.mul_El = small_div_mul(a.E / a.R); a.mul_K = small_div_mul(a.K);
    a.tpc = plan.tpc; a.n_groups = ceil_div(a.T, 32); a.vec_per_row = shape->hidden / 8; a.wpr = plan.wpr;
    layout_dispatch_small_kernel<<<plan.n_ctas, kFusedThreads, plan.smem, stream>>>(a);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}
