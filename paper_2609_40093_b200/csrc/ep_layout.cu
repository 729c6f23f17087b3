// ep_layout: counts, prefix scans and deterministic destination slots, all on the device.
//
// The work is a stable counting sort of the T*K (token, k) pairs by expert id plus
// a stable count of the distinct (token, rank) hits. Determinism never depends on
// the arrival order of atomics between warps: tokens are cut into contiguous tiles
// of 32*m tokens, one warp owns a tile, a CTA owns `warps` consecutive tiles, and
// every rank inside a tile comes from warp ballots / matches whose lane order is
// the (t,k) order. Every CTA
//   1. histograms its tiles (experts, rank hits, bad ids) in shared memory, one
//      private histogram per warp,
//   2. learns, per bin, the count in earlier CTAs and the grand total,
//   3. scans the totals over bins (expert_offsets, rank_row_offsets),
//   4. replays its tiles in (t,k) order with running counters that start at
//      offset[bin] + earlier CTAs + earlier warps of this CTA.
// Step 2 has three forms:
//   single   one CTA of up to 8 warps holds every tile (up to 256 tokens): nothing
//            to exchange, one launch (32 warps on one SM took 26 us for 1024 tokens,
//            four CTAs of 8 warps take 12);
//   cluster  up to 8 CTAs of 8 warps (up to 2048 tokens) form one thread-block cluster
//            and read each other's CTA totals through distributed shared memory
//            between two cluster barriers: one launch, no global scratch;
//   global   larger batches, or a device that cannot keep the cluster resident: up to
//            128 CTAs of 8 warps, because the replay's scattered 4-byte stores (two per
//            pair) are bound per SM (at T=8192, K=8: 8 CTAs of 32 warps 24 us, 32 CTAs of
//            8 warps 15 us); a first kernel writes cta_part[cta][bin] to the
//            workspace; the main kernel, launched with programmatic stream
//            serialisation so that its histogram phase overlaps the first kernel,
//            executes griddepcontrol.wait and then reads every cta_part row.
// Bins: [0,E) experts, [E,E+R) rank hits, [E+R] ids outside [-1,E).
//
// Inner loops: the ids of 32 tokens are staged in shared memory with an odd row
// stride (token-per-lane and pair-per-lane accesses are both free of bank
// conflicts); divisions by E/R and K are one 32-bit high multiply; a rank's ballot
// is kept by lane r, so the R ballots of a group cost R votes and no serial
// section; the running counter of an expert is advanced by one shared-memory
// atomic of the group's first lane (the counters are private to the warp, so their
// order is the program order of that warp).
#include <cooperative_groups.h>

#include <atomic>
#include <mutex>

#include "ep_common.cuh"
#include "ep_layout_common.cuh"

namespace cg = cooperative_groups;

namespace ep {
namespace {

constexpr int kMaxWarpsSingle = 8;      // one CTA holds every tile: up to 256 tokens
constexpr int kMaxWarps = 8;            // warps per CTA otherwise (the replay's scattered stores are bound per SM: spread it)
constexpr int kMaxCluster = 8;          // portable cluster size
constexpr int kMaxCtasGlobal = 128;
constexpr size_t kSmemBudget = 200 * 1024;
constexpr int kSteps = 2;               // 32-pair steps of the replay whose latencies overlap (4 in flight: 1 us slower at T=8192)

enum { kModeSingle = 0, kModeCluster = 1, kModeGlobal = 2 };
enum { kPartRanks = 1, kPartPairs = 2 };
constexpr int kLeanTokensPerCta = 256;              // the lean kernels: 8 warps, one token per lane
constexpr int kLeanMaxCtas = 128;
constexpr int kLeanMaxExperts = 1024;

struct LayoutPlan {
    int mode;
    int tile_tokens;    // tokens per tile, a multiple of 32
    int n_tiles;
    int bins;           // E + R + 1
    int warps;          // tiles per CTA
    int n_ctas;
    size_t smem;        // dynamic shared memory
    size_t workspace_bytes;
};

// shared memory: per warp  hist[bins] | ballots[kMaxRanks] | rows[32][Kp] | ids[32][Kp]   (Kp = K | 1);
//                per CTA   tot[bins+1] | pre[bins] | cta_tot[bins] | scan[32]
inline size_t per_warp_ints(int bins, int K) { return (size_t)bins + kMaxRanks + 64 * (size_t)(K | 1); }
inline size_t per_cta_ints(int bins) { return 3 * (size_t)bins + 2 + 32; }

LayoutPlan make_plan(const ep_shape_t &s)
{
    LayoutPlan p;
    const int T = s.num_tokens > 0 ? s.num_tokens : 1;
    p.bins = s.num_experts + s.num_ranks + 1;
    const size_t pw = sizeof(int32_t) * per_warp_ints(p.bins, s.top_k), pc = sizeof(int32_t) * per_cta_ints(p.bins);
    int fit = (int)((kSmemBudget - pc) / pw);
    fit = fit < 1 ? 1 : fit;
    const int groups = ceil_div(T, 32);                 // 32-token groups
    const int w1 = fit > kMaxWarpsSingle ? kMaxWarpsSingle : fit;
    const int w = fit > kMaxWarps ? kMaxWarps : fit;
    if (groups <= w1) {
        p.mode = kModeSingle;
        p.tile_tokens = 32;
        p.n_tiles = groups;
        p.warps = groups;
        p.n_ctas = 1;
    } else {
        p.tile_tokens = 32 * ceil_div(groups, kMaxCtasGlobal * w);
        p.n_tiles = ceil_div(T, p.tile_tokens);
        p.warps = w;
        p.n_ctas = ceil_div(p.n_tiles, w);
        p.mode = p.n_ctas <= kMaxCluster ? kModeCluster : kModeGlobal;
    }
    p.smem = pw * p.warps + pc;
    // the cluster form needs no scratch, but falls back to the global form on a device that cannot
    // keep the whole cluster resident, so both ask for cta_part
    p.workspace_bytes = p.mode == kModeSingle ? 16 : sizeof(int32_t) * (size_t)p.n_ctas * p.bins;
    // the lean kernel pair (256 tokens per CTA) takes over from 257 tokens on: one scratch row per CTA of its own
    const int lean_ctas = ceil_div(T, kLeanTokensPerCta);
    if (lean_ctas > 1 && lean_ctas <= kLeanMaxCtas) {
        const size_t lean = sizeof(int32_t) * (size_t)lean_ctas * p.bins;
        p.workspace_bytes = lean > p.workspace_bytes ? lean : p.workspace_bytes;
    }
    return p;
}

struct LayoutArgs {
    const int32_t *idx;
    ep_layout_t out;
    int32_t *cta_part;  // [n_ctas][bins], global form only
    int T, top_k, E, num_ranks, Tr;
    uint32_t mul_El, mul_K, mul_R1;   // multipliers of sdiv for E/R, K and R+1
    FastDiv by_Tr;
    int tile_tokens, n_tiles, bins, n_ctas, mode;
    int parts;   // kPartRanks | kPartPairs: which outputs this call writes
    int blo;     // first bin in use: 0, or E when only the receive-row half is wanted
};

// The warp copies the expert ids of the 32 tokens [tb, tb+32) into ids[32][Kp] (coalesced, eight loads
// per lane in flight before the first use); entries of tokens >= t1 become -1. Returns the number of live items.
template <int KT>
__device__ __forceinline__ int stage_group(const LayoutArgs &a, int32_t *ids, int tb, int t1, int lane)
{
    const int K = KT ? KT : a.top_k, Kp = K | 1;
    const int n_items = (min(t1, tb + 32) - tb) * K;
    const int32_t *src = a.idx + (size_t)tb * K;
    for (int base = lane; base < 32 * K; base += 256) {
        int32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + 32 * u;
            v[u] = i < n_items ? __ldg(src + i) : -1;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = base + 32 * u;
            if (i < 32 * K) {
                const int tok = sdiv(i, a.mul_K);
                ids[tok * Kp + (i - tok * K)] = v[u];
            }
        }
    }
    __syncwarp();
    return n_items;
}

// position in ids[] / rows[] of pair i (in (t,k) order) of the staged group
template <int KT>
__device__ __forceinline__ int pair_pos(const LayoutArgs &a, int i)
{
    const int K = KT ? KT : a.top_k, Kp = K | 1;
    const int tok = sdiv(i, a.mul_K);
    return tok * Kp + (i - tok * K);
}

// rank bitmask of the token this lane owns in the staged group; *bad counts ids outside [-1, E)
template <int KT>
__device__ __forceinline__ unsigned long long token_rank_mask(const LayoutArgs &a, const int32_t *ids, int lane, int *bad)
{
    const int K = KT ? KT : a.top_k, Kp = K | 1;
    unsigned long long mask = 0ull;
    for (int k = 0; k < K; ++k) {
        const int e = ids[lane * Kp + k];
        if (e >= 0 && e < a.E) mask |= 1ull << sdiv(e, a.mul_El);
        else if (e != -1) ++*bad;
    }
    return mask;
}

// One warp counts its tile into hist[bins]. kShared == false: hist is this warp's own and is
// zeroed here; kShared == true: hist is one histogram for the whole CTA, zeroed by the caller.
// Returns the rank mask of this lane's token in the tile's last group (reused by a one-group replay).
template <bool kShared, int KT, int RT>
__device__ __forceinline__ unsigned long long count_tile(const LayoutArgs &a, int32_t *hist, int32_t *ids, int tile, int lane)
{
    const int K = KT ? KT : a.top_k, Kp = K | 1, R = RT ? RT : a.num_ranks;
    if (!kShared) {
        for (int b = a.blo + lane; b < a.bins; b += 32) hist[b] = 0;
        __syncwarp();
    }
    if (tile >= a.n_tiles) return 0ull;
    const int t0 = tile * a.tile_tokens;
    const int t1 = min(a.T, t0 + a.tile_tokens);
    int bad = 0;
    int hits0 = 0, hits1 = 0;                        // lane l counts the hits of ranks l and l + 32
    unsigned long long mask = 0ull;
    for (int tb = t0; tb < t1; tb += 32) {
        stage_group<KT>(a, ids, tb, t1, lane);
        if (a.blo == 0)                               // experts: any order
            for (int k = 0; k < K; ++k) {
                const int e = ids[lane * Kp + k];
                if (e >= 0 && e < a.E) atomicAdd(hist + e, 1);
            }
        mask = token_rank_mask<KT>(a, ids, lane, &bad);   // rank hits: token per lane, ballot per rank
        for (int r = 0; r < R; ++r) {
            const int c = __popc(__ballot_sync(kFullMask, (mask >> r) & 1ull));
            if (lane == (r & 31)) {
                if (r < 32) hits0 += c;
                else hits1 += c;
            }
        }
        __syncwarp();
    }
    if (kShared) {
        if (lane < R && hits0) atomicAdd(hist + a.E + lane, hits0);
        if (lane + 32 < R && hits1) atomicAdd(hist + a.E + 32 + lane, hits1);
    } else {
        if (lane < R) hist[a.E + lane] = hits0;
        if (lane + 32 < R) hist[a.E + 32 + lane] = hits1;
    }
    if (bad) atomicAdd(hist + a.E + R, bad);
    __syncwarp();
    return mask;
}

// ---------------------------------------------------------------- global form, first kernel
template <int KT, int RT>
__global__ void __launch_bounds__(kMaxWarps * 32) layout_cta_count_kernel(LayoutArgs a)
{
    const int K = KT ? KT : a.top_k, Kp = K | 1;
    pdl_trigger();                                                    // the main kernel may start its own counting now
    extern __shared__ int32_t smem[];
    const int warps = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // one histogram for the CTA (first `bins` words), per-warp id staging behind it
    for (int b = a.blo + threadIdx.x; b < a.bins; b += blockDim.x) smem[b] = 0;
    __syncthreads();
    count_tile<true, KT, RT>(a, smem, smem + a.bins + warp * 32 * Kp, blockIdx.x * warps + warp, lane);
    __syncthreads();
    int32_t *dst = a.cta_part + (size_t)blockIdx.x * a.bins;
    for (int b = a.blo + threadIdx.x; b < a.bins; b += blockDim.x) dst[b] = smem[b];
}

// ---------------------------------------------------------------- main kernel
template <int KT, int RT>
__global__ void __launch_bounds__(kMaxWarpsSingle * 32) layout_assign_kernel(LayoutArgs a)
{
    const int K = KT ? KT : a.top_k, Kp = K | 1, R = RT ? RT : a.num_ranks;
    pdl_trigger();     // a kernel launched behind this one with programmatic serialisation may become resident
    extern __shared__ int32_t smem[];
    const int warps = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pw = a.bins + kMaxRanks + 64 * Kp;
    const int nb = a.E + R;
    int32_t *run = smem + warp * pw;                                 // [bins] histogram, later next free slot
    unsigned *bal = reinterpret_cast<unsigned *>(run + a.bins);      // [R] ballots of the current 32 tokens
    int32_t *rows = run + a.bins + kMaxRanks;                        // [32][Kp] receive rows of the current 32 tokens
    int32_t *ids = rows + 32 * Kp;                                 // [32][Kp] expert ids of the current 32 tokens
    int32_t *tot = smem + warps * pw;                                // [E+R+1] totals -> one scan: experts, then ranks
    int32_t *pre = tot + a.bins + 1;                                 // [bins] count in earlier CTAs
    int32_t *cta_tot = pre + a.bins;                                 // [bins] this CTA's totals (peers read it)
    int32_t *sh = cta_tot + a.bins;                                  // [32] scan scratch
    const int tile = blockIdx.x * warps + warp;
    const unsigned lt = lanemask_lt();

    const unsigned long long mask_kept = count_tile<false, KT, RT>(a, run, ids, tile, lane);
    __syncthreads();
    const bool ranks = a.parts & kPartRanks, pairs = a.parts & kPartPairs;
    for (int b = a.blo + threadIdx.x; b < a.bins; b += blockDim.x) {  // this CTA's total per bin
        int32_t mine = 0;
#pragma unroll 8
        for (int w = 0; w < warps; ++w) mine += smem[w * pw + b];
        cta_tot[b] = mine;
    }
    if (a.mode == kModeCluster) cg::this_cluster().sync();           // every peer's cta_tot is written
    else if (a.mode == kModeGlobal) pdl_wait();                      // cta_part is complete and visible
    // per bin: count in earlier CTAs and grand total (each thread reads the cta_tot entries it wrote itself)
    for (int b = a.blo + threadIdx.x; b < a.bins; b += blockDim.x) {
        int32_t before = 0, total = 0;
        if (a.mode == kModeCluster) {
            cg::cluster_group cluster = cg::this_cluster();
#pragma unroll 8
            for (int c = 0; c < a.n_ctas; ++c) {
                const int32_t v = cluster.map_shared_rank(cta_tot, c)[b];
                total += v;
                if (c < (int)blockIdx.x) before += v;
            }
        } else if (a.mode == kModeGlobal) {
            column_sums<16>(a.cta_part + b, a.bins, a.n_ctas, blockIdx.x, a.T < 0, a.cta_part, &total, &before);
        } else {
            total = cta_tot[b];
        }
        pre[b] = before;
        if (b < nb) tot[b] = total;
        if (blockIdx.x == 0) {
            if (b < a.E) a.out.expert_counts[b] = total;               // only reached when the pair half is wanted
            else if (!ranks) continue;
            else if (b < nb) a.out.rank_rows[b - a.E] = total;
            else *a.out.status = total ? EP_STATUS_BAD_INDEX : 0;
        }
    }
    if (a.mode == kModeCluster) cg::this_cluster().sync();           // peers are done with this CTA's shared memory
    else __syncthreads();
    // one exclusive scan over [experts | ranks]: S[e] = expert offset, S[E + r] - S[E] = rank row offset
    block_exclusive_scan_smem(tot + a.blo, nb - a.blo, sh);
    const int32_t n_pairs = tot[a.E];                                // 0 when the scan started at the rank bins
    if (blockIdx.x == 0) {
        if (pairs)
            for (int e = threadIdx.x; e <= a.E; e += blockDim.x) a.out.expert_offsets[e] = tot[e];
        if (ranks) {
            for (int r = threadIdx.x; r <= R; r += blockDim.x) a.out.rank_row_offsets[r] = tot[a.E + r] - n_pairs;
            for (int r = threadIdx.x; r < R; r += blockDim.x)
                a.out.src_row_offsets[r * (R + 1) + R] = tot[a.E + r + 1] - n_pairs;
        }
    }
    // next free slot of every bin for every warp: offset + earlier CTAs + earlier warps of this CTA
    for (int b = a.blo + threadIdx.x; b < nb; b += blockDim.x) {
        int32_t running = pre[b] + (b < a.E ? tot[b] : tot[b] - n_pairs);
        for (int w0 = 0; w0 < warps; w0 += 8) {                      // eight counts read before the first is replaced
            int32_t v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = w0 + u < warps ? smem[(w0 + u) * pw + b] : 0;
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (w0 + u < warps) {
                    smem[(w0 + u) * pw + b] = running;
                    running += v[u];
                }
        }
    }
    __syncthreads();
    if (tile >= a.n_tiles) return;

    // replay the tile in (t,k) order; run[bin] = next free slot of the bin
    const int t0 = tile * a.tile_tokens;
    const int t1 = min(a.T, t0 + a.tile_tokens);
    for (int tb = t0; tb < t1; tb += 32) {
        const int t = tb + lane;
        const bool live = t < t1;
        // a tile of one 32-token group still has its ids staged (and its rank masks) from the counting phase
        int n_items, bad = 0;
        unsigned long long mask;
        if (a.tile_tokens == 32) {
            n_items = (min(t1, tb + 32) - tb) * K;
            mask = mask_kept;
        } else {
            n_items = stage_group<KT>(a, ids, tb, t1, lane);
            mask = token_rank_mask<KT>(a, ids, lane, &bad);
        }
        // --- receive rows: which of these 32 tokens hit which rank (lane r keeps rank r's ballot)
        for (int r = 0; r < R; ++r) {
            const unsigned b = __ballot_sync(kFullMask, (mask >> r) & 1ull);
            if (lane == (r & 31)) bal[r] = b;
        }
        __syncwarp();
        if (live) {
            const int s = fdiv(t, a.by_Tr);
            if (ranks && t == s * a.Tr)              // first token of source rank s
                for (int r = 0; r < R; ++r)
                    a.out.src_row_offsets[r * (R + 1) + s] = run[a.E + r] + __popc(bal[r] & lt);
            for (int k = 0; k < K; ++k) {
                const int e = ids[lane * Kp + k];
                int32_t row = -1;
                if (e >= 0 && e < a.E) {
                    const int r = sdiv(e, a.mul_El);
                    row = run[a.E + r] + __popc(bal[r] & lt);
                }
                rows[lane * Kp + k] = row;
            }
        }
        // receive row -> token, rank by rank: the tokens of these 32 that hit rank r own consecutive rows, so
        // each rank costs one store to one or two cache lines (a store per pick would touch a line per rank)
        if (ranks)
            for (int r = 0; r < R; ++r)
                if (live && ((mask >> r) & 1ull)) a.out.recv_token[run[a.E + r] + __popc(bal[r] & lt)] = t;
        __syncwarp();
        for (int r = lane; r < R; r += 32) run[a.E + r] += __popc(bal[r]);
        __syncwarp();
        int32_t *recv_slot = a.out.recv_slot + (size_t)tb * K;
        if (!pairs) {                                // receive-row half only: publish the rows and go on
            for (int i = lane; i < n_items; i += 32) recv_slot[i] = rows[pair_pos<KT>(a, i)];
            __syncwarp();
            continue;
        }
        // --- pair slots: the items of these tokens, 32 at a time in (t,k) order
        int32_t *pair_slot = a.out.pair_slot + (size_t)tb * K;
        for (int j0 = 0; j0 < n_items; j0 += 32 * kSteps) {          // kSteps steps of 32 pairs: their matches, then their
            int pos[kSteps], e[kSteps], leader[kSteps];              // counter updates in order, then their stores
            unsigned m[kSteps];
            int32_t first[kSteps];
#pragma unroll
            for (int u = 0; u < kSteps; ++u) {
                const int i = j0 + 32 * u + lane;
                const int tok = sdiv(i, a.mul_K);
                pos[u] = tok * Kp + (i - tok * K);
                e[u] = i < n_items ? ids[pos[u]] : -1;
                if (e[u] >= a.E) e[u] = -2;                          // out of range: masked like any negative id
            }
#pragma unroll
            for (int u = 0; u < kSteps; ++u) {
                m[u] = __match_any_sync(kFullMask, e[u] >= 0 ? e[u] : a.E + lane);
                leader[u] = __ffs(m[u]) - 1;
            }
#pragma unroll
            for (int u = 0; u < kSteps; ++u) {
                first[u] = 0;
                if (e[u] >= 0 && lane == leader[u]) first[u] = atomicAdd(run + e[u], __popc(m[u]));   // the group's slots at once
                __syncwarp();                        // orders this step's counter update before the next step's
            }
#pragma unroll
            for (int u = 0; u < kSteps; ++u) {
                const int i = j0 + 32 * u + lane;
                first[u] = __shfl_sync(kFullMask, first[u], leader[u]);
                if (e[u] >= 0) {
                    const int32_t p = first[u] + __popc(m[u] & lt);
                    const int32_t row = rows[pos[u]];
                    pair_slot[i] = p;
                    if (ranks) recv_slot[i] = row;
                    a.out.pair_token[p] = tb + sdiv(i, a.mul_K);
                    a.out.pair_row[p] = row;
                } else if (i < n_items) {
                    pair_slot[i] = -1;
                    if (ranks) recv_slot[i] = -1;
                }
            }
        }
    }
}

}  // namespace
}  // namespace ep

extern "C" size_t ep_layout_workspace_bytes(const ep_shape_t *shape)
{
    if (ep::check_shape(shape, false) != EP_OK) return 0;
    return ep::make_plan(*shape).workspace_bytes;
}

namespace ep {
namespace {

// ---------------------------------------------------------------- lean form
// Compile-time K (1..8 and 10), a compile-time bound RT on the ranks (8, 16, 32 or 64; 64 is the library's limit) and, for
// the pair half, E <= 1024: one token per lane
// with its picks in registers (vector loads, no staging for the counting), the rank ballots in registers, 256
// tokens per CTA. Up to 256 tokens the main kernel runs alone as one CTA (its own counters are the totals). Beyond,
// the same two-kernel exchange as the general form: the first kernel writes
// cta_part[cta] = [R rank-hit counters | bad ids | E expert counters], the second is launched with programmatic
// stream serialisation and waits on the device before it reads them: it requests its share of the rank counters
// and then a batch of expert counters (one expert per thread) before it uses either, so that both exchanges share
// one L2 round trip (the rank counters are summed by shared-memory atomics: only sums are used). In the receive-row
// half every warp scans the ranks itself and sets its own receive-row bases; in the pair half one warp does that
// for all while another scans the experts. Every pick's receive row is looked up by its rank; the slots leave as
// 16-byte stores. The pair half replays each warp's 32*K pairs in (t,k) order from a staged copy, two 32-pair
// steps in flight, with warp-private expert counters as in the general form.
//   PAIRS == false: the receive-row half alone (what dispatch waits for), no dynamic shared memory;
//   PAIRS == true : the pair half, or both halves (a.parts).
constexpr int kLeanWarps = kLeanTokensPerCta / 32;
constexpr int kLeanSteps = 2;                     // 32-pair steps of the replay in flight (8.3 us per call at C4; 8.9 with 1, 9.6 with 4, 10.4 with 8)
constexpr int kLeanExchangeBatch = 32;              // CTAs' expert counters a thread requests at once

inline size_t lean_smem_bytes(int E, int K)
{
    // ids_s[W][32*K] | rows_s[W][32*K] | whist[W][E] | tot[E+1] | before[E] | scan[32]
    return sizeof(int32_t) * ((size_t)kLeanWarps * E + (E + 1) + E + 2 * (size_t)kLeanWarps * 32 * K + 32);
}

template <int KT>
__device__ __forceinline__ void load_picks(const int32_t *idx, int t, int32_t (&e)[KT])
{
    if (KT % 4 == 0) {
        const int4 *p = reinterpret_cast<const int4 *>(idx + (size_t)t * KT);
#pragma unroll
        for (int i = 0; i < KT / 4; ++i) {
            const int4 v = __ldg(p + i);
            e[4 * i] = v.x; e[4 * i + 1] = v.y; e[4 * i + 2] = v.z; e[4 * i + 3] = v.w;
        }
    } else if (KT % 2 == 0) {
        const int2 *p = reinterpret_cast<const int2 *>(idx + (size_t)t * KT);
#pragma unroll
        for (int i = 0; i < KT / 2; ++i) {
            const int2 v = __ldg(p + i);
            e[2 * i] = v.x; e[2 * i + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < KT; ++i) e[i] = __ldg(idx + (size_t)t * KT + i);
    }
}

// KT ints of one token to global or shared memory as 16- or 8-byte stores (odd KT: one by one)
template <int KT>
__device__ __forceinline__ void store_picks(int32_t *dst, const int32_t (&v)[KT])
{
    if (KT % 4 == 0) {
#pragma unroll
        for (int i = 0; i < KT / 4; ++i)
            reinterpret_cast<int4 *>(dst)[i] = make_int4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else if (KT % 2 == 0) {
#pragma unroll
        for (int i = 0; i < KT / 2; ++i) reinterpret_cast<int2 *>(dst)[i] = make_int2(v[2 * i], v[2 * i + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < KT; ++i) dst[i] = v[i];
    }
}

// rank bitmask of a token: 32 bits up to 32 ranks, 64 beyond
template <int RT>
struct RankMask {
    using type = unsigned;
};
template <>
struct RankMask<64> {
    using type = unsigned long long;
};

// picks -> ranks (or -1), rank bitmask, number of ids outside [-1, E)
template <int KT, typename Mask>
__device__ __forceinline__ Mask picks_to_ranks(const LayoutArgs &a, const int32_t (&e)[KT], int (&rk)[KT], int *bad)
{
    Mask mask = 0;
#pragma unroll
    for (int k = 0; k < KT; ++k) {
        rk[k] = -1;
        if ((unsigned)e[k] < (unsigned)a.E) {
            rk[k] = sdiv(e[k], a.mul_El);
            mask |= Mask(1) << rk[k];
        } else if (e[k] != -1) {
            ++*bad;
        }
    }
    return mask;
}

template <int KT, int RT, bool PAIRS>
__global__ void __launch_bounds__(kLeanWarps * 32) lean_count_kernel(LayoutArgs a)
{
    pdl_trigger();                                   // the second kernel may start its own loads now
    extern __shared__ int32_t dyn[];                 // PAIRS: this CTA's expert histogram [E]
    __shared__ int32_t cnt[RT + 1];
    const int tid = threadIdx.x, lane = tid & 31;
    const int t = blockIdx.x * (kLeanWarps * 32) + tid;
    if (tid <= RT) cnt[tid] = 0;
    if (PAIRS)
        for (int x = tid; x < a.E; x += kLeanWarps * 32) dyn[x] = 0;
    int32_t e[KT];
    int rk[KT], bad = 0;
#pragma unroll
    for (int k = 0; k < KT; ++k) e[k] = -1;
    if (t < a.T) load_picks<KT>(a.idx, t, e);
    using Mask = typename RankMask<RT>::type;
    constexpr int kRanksPerLane = (RT + 31) / 32;    // lane l counts ranks l, l + 32
    const Mask mask = picks_to_ranks<KT, Mask>(a, e, rk, &bad);
    __syncthreads();
    if (PAIRS) {
#pragma unroll
        for (int k = 0; k < KT; ++k)
            if (rk[k] >= 0) atomicAdd(dyn + e[k], 1);
    }
    int mine[kRanksPerLane] = {};
#pragma unroll
    for (int r = 0; r < RT; ++r) {
        const int c = __popc(__ballot_sync(kFullMask, (unsigned)(mask >> r) & 1u));
        if (lane == (r & 31)) mine[r >> 5] = c;
    }
#pragma unroll
    for (int j = 0; j < kRanksPerLane; ++j)
        if (lane + 32 * j < RT && mine[j]) atomicAdd(cnt + lane + 32 * j, mine[j]);
    if (bad) atomicAdd(cnt + RT, bad);
    __syncthreads();
    // one row per CTA, as wide as the general form's: [R rank-hit counters | bad ids | E expert counters]
    const int R = a.num_ranks;
    int32_t *row = a.cta_part + (size_t)blockIdx.x * (R + 1 + (PAIRS ? a.E : 0));
    if (tid < R) row[tid] = cnt[tid];
    if (tid == RT) row[R] = cnt[RT];
    if (PAIRS)
        for (int x = tid; x < a.E; x += kLeanWarps * 32) row[R + 1 + x] = dyn[x];
}

template <int KT, int RT, bool PAIRS>
__global__ void __launch_bounds__(kLeanWarps * 32) lean_assign_kernel(LayoutArgs a)
{
    pdl_trigger();
    extern __shared__ int32_t dyn[];
    __shared__ int32_t wcnt[kLeanWarps][RT];         // rank hits per warp
    __shared__ int32_t base[kLeanWarps][RT];         // first receive row of each warp's tokens per rank
    __shared__ unsigned bal_s[kLeanWarps][RT];       // which of a warp's 32 tokens hit rank r
    __shared__ int32_t acc[2][RT + 1];               // per rank (and bad ids): hits in earlier CTAs, hits in all
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tw = blockIdx.x * (kLeanWarps * 32) + warp * 32;   // this warp's first token
    const int t = tw + lane;
    const unsigned lt = lanemask_lt();
    const int E = a.E, R = a.num_ranks, stride = R + 1 + (PAIRS ? E : 0);    // R <= RT: ranks R..RT-1 are never hit
    const bool ranks = !PAIRS || (a.parts & kPartRanks);
    // PAIRS: ids_s[W][32*KT] | rows_s[W][32*KT] (both written by 16-byte stores) | whist[W][E] | tot[E+1] | before[E] | scan[32]
    int32_t *ids_s = dyn + warp * 32 * KT;
    int32_t *rows_s = dyn + kLeanWarps * 32 * KT + warp * 32 * KT;
    int32_t *hist = dyn + 2 * kLeanWarps * 32 * KT;  // [W][E]
    int32_t *whist = hist + warp * E;                // this warp's expert counts, later next free pair slot
    int32_t *tot = hist + kLeanWarps * E;
    int32_t *before_e = tot + E + 1;
    int32_t *sh = before_e + E;

    int32_t e[KT];
    int rk[KT], bad = 0;
#pragma unroll
    for (int k = 0; k < KT; ++k) e[k] = -1;
    if (t < a.T) load_picks<KT>(a.idx, t, e);
    using Mask = typename RankMask<RT>::type;
    constexpr int kRanksPerLane = (RT + 31) / 32;    // lane l scans ranks l, l + 32
    constexpr bool kKeepBallots = RT <= 32;          // the ballots stay in registers too, or only in shared memory
    const Mask mask = picks_to_ranks<KT, Mask>(a, e, rk, &bad);
    unsigned bal[kKeepBallots ? RT : 1];
#pragma unroll
    for (int r = 0; r < RT; ++r) {
        const unsigned b = __ballot_sync(kFullMask, (unsigned)(mask >> r) & 1u);
        if (kKeepBallots) bal[kKeepBallots ? r : 0] = b;
        if (lane == (r & 31)) {
            wcnt[warp][r] = __popc(b);
            bal_s[warp][r] = b;
        }
    }
    if (PAIRS) {
        for (int x = lane; x < E; x += 32) whist[x] = 0;
        store_picks<KT>(ids_s + lane * KT, e);       // the warp's pairs in (t,k) order
        __syncwarp();
#pragma unroll
        for (int k = 0; k < KT; ++k)
            if (rk[k] >= 0) atomicAdd(whist + e[k], 1);
    }
    if (tid < 2 * (RT + 1)) (&acc[0][0])[tid] = 0;
    __syncthreads();
    if (a.mode == kModeSingle) {
        // one CTA holds the whole batch (at most 256 tokens): its own counters are the totals; no first kernel, no scratch
        if (tid < RT) {
            int32_t hits = 0;
#pragma unroll
            for (int w = 0; w < kLeanWarps; ++w) hits += wcnt[w][tid];
            acc[1][tid] = hits;
        }
        if (bad) atomicAdd(&acc[1][RT], bad);
        if (PAIRS) {
            for (int x = tid; x < E; x += kLeanWarps * 32) {
                int32_t total = 0;
#pragma unroll
                for (int w = 0; w < kLeanWarps; ++w) total += hist[w * E + x];
                tot[x] = total;
                before_e[x] = 0;
                a.out.expert_counts[x] = total;
            }
        }
    } else {
        pdl_wait();                                      // cta_part is complete and visible
        // rank counters of every CTA: the first kRankBatch per thread are requested here and summed (shared-memory
        // atomics) behind the expert counters' batch, so that both exchanges share one L2 round trip
        constexpr int kRankBatch = RT <= 8 ? 2 : RT <= 16 ? 3 : RT <= 32 ? 5 : 9;    // 32 CTAs x (RT + 1) counters over 256 threads
        const int n_items = a.n_ctas * (R + 1);
        int32_t rv[kRankBatch];
        int rc[kRankBatch], rr[kRankBatch];
#pragma unroll
        for (int u = 0; u < kRankBatch; ++u) {
            const int i = min(tid + u * kLeanWarps * 32, n_items - 1);
            rc[u] = sdiv(i, a.mul_R1);
            rr[u] = i - rc[u] * (R + 1);
            rv[u] = __ldcg(a.cta_part + (size_t)rc[u] * stride + rr[u]);
        }
        if (!PAIRS && a.T < 0 && tid == 0) *a.cta_part = (int32_t)clock64();   // never true: ends the basic block (see column_sums)
        if (PAIRS) {                                     // expert counters: one expert per thread, coalesced rows
            for (int x = tid; x < E; x += kLeanWarps * 32) {
                int32_t before, total;
                const int32_t *col = a.cta_part + R + 1 + x;
                if (a.n_ctas <= 16) column_sums<16>(col, stride, a.n_ctas, blockIdx.x, a.T < 0, a.cta_part, &total, &before);
                else column_sums<kLeanExchangeBatch>(col, stride, a.n_ctas, blockIdx.x, a.T < 0, a.cta_part, &total, &before);
                tot[x] = total;
                before_e[x] = before;
                if (blockIdx.x == 0) a.out.expert_counts[x] = total;
            }
        }
#pragma unroll
        for (int u = 0; u < kRankBatch; ++u) {
            const int slot = rr[u] < R ? rr[u] : RT;     // the counter behind the ranks holds the bad ids
            if (tid + u * kLeanWarps * 32 < n_items && rv[u]) {
                atomicAdd(&acc[1][slot], rv[u]);
                if (rc[u] < (int)blockIdx.x) atomicAdd(&acc[0][slot], rv[u]);
            }
        }
        for (int i = tid + kRankBatch * kLeanWarps * 32; i < n_items; i += kLeanWarps * 32) {    // more counters: the rest
            const int c = sdiv(i, a.mul_R1), r = i - c * (R + 1);
            const int32_t v = __ldcg(a.cta_part + (size_t)c * stride + r);
            const int slot = r < R ? r : RT;
            if (v) {
                atomicAdd(&acc[1][slot], v);
                if (c < (int)blockIdx.x) atomicAdd(&acc[0][slot], v);
            }
        }
    }
    __syncthreads();
    // PAIRS: warp 1 scans the ranks and sets every warp's bases while warp 0 scans the experts. Otherwise every warp
    // scans the ranks itself and sets its own bases: no serial section, no second block barrier.
    if (!PAIRS || warp == 1) {
        // lane l: ranks l and (RT = 64) l + 32; acc[.][RT] holds the ids outside [-1, E)
        int32_t before[kRanksPerLane], hits[kRanksPerLane], incl[kRanksPerLane];
        int32_t carry = 0;                           // hits of the ranks below this lane's j-th rank's block of 32
#pragma unroll
        for (int j = 0; j < kRanksPerLane; ++j) {
            const int r = lane + 32 * j;
            before[j] = r < R ? acc[0][r] : 0;
            hits[j] = r < R ? acc[1][r] : 0;
            int32_t x = hits[j];                     // scan over ranks: rank_row_offsets
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t up = __shfl_up_sync(kFullMask, x, off);
                if (lane >= off) x += up;
            }
            incl[j] = x + carry;
            carry = __shfl_sync(kFullMask, incl[j], 31);
        }
        const int32_t n_recv = carry;
        if (blockIdx.x == 0 && ranks && (PAIRS || warp == 0)) {
#pragma unroll
            for (int j = 0; j < kRanksPerLane; ++j) {
                const int r = lane + 32 * j;
                if (r < R) {
                    a.out.rank_rows[r] = hits[j];
                    a.out.rank_row_offsets[r] = incl[j] - hits[j];
                    a.out.src_row_offsets[r * (R + 1) + R] = incl[j];
                }
            }
            if (lane == 0) {
                a.out.rank_row_offsets[R] = n_recv;
                *a.out.status = acc[1][RT] ? EP_STATUS_BAD_INDEX : 0;
            }
        }
#pragma unroll
        for (int j = 0; j < kRanksPerLane; ++j) {
            const int r = lane + 32 * j;
            if (r < RT) {
                int32_t run = incl[j] - hits[j] + before[j];
                if (PAIRS) {
#pragma unroll
                    for (int w = 0; w < kLeanWarps; ++w) {
                        base[w][r] = run;
                        run += wcnt[w][r];
                    }
                } else {
#pragma unroll
                    for (int w = 0; w < kLeanWarps - 1; ++w) run += w < warp ? wcnt[w][r] : 0;
                    base[warp][r] = run;
                }
            }
        }
    }
    if (PAIRS) {
        block_exclusive_scan_smem(tot, E, sh);       // tot[x] = expert offset, tot[E] = number of pairs
        for (int x = tid; x < E; x += kLeanWarps * 32) {   // next free pair slot of expert x for every warp
            int32_t run = tot[x] + before_e[x];
#pragma unroll
            for (int w = 0; w < kLeanWarps; ++w) {
                const int32_t c = hist[w * E + x];
                hist[w * E + x] = run;
                run += c;
            }
        }
        if (blockIdx.x == 0)
            for (int x = tid; x <= E; x += kLeanWarps * 32) a.out.expert_offsets[x] = tot[x];
        __syncthreads();
    } else {
        __syncwarp();
    }
    const bool live = t < a.T;
    int32_t rows[KT];                                // receive row of every pick: looked up by its rank
#pragma unroll
    for (int k = 0; k < KT; ++k) rows[k] = rk[k] >= 0 ? base[warp][rk[k]] + __popc(bal_s[warp][rk[k]] & lt) : -1;
    if (ranks && live) {
        store_picks<KT>(a.out.recv_slot + (size_t)t * KT, rows);
        const int s = fdiv(t, a.by_Tr);
        const bool first_of_source = t == s * a.Tr;  // where source rank s's segment starts in every rank
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            const int32_t row = base[warp][r] + __popc((kKeepBallots ? bal[kKeepBallots ? r : 0] : bal_s[warp][r]) & lt);
            if ((unsigned)(mask >> r) & 1u) a.out.recv_token[row] = t;   // a rank's rows of these 32 tokens are consecutive
            if (first_of_source && r < R) a.out.src_row_offsets[r * (R + 1) + s] = row;
        }
    }
    if (!PAIRS) return;
    store_picks<KT>(rows_s + lane * KT, rows);
    __syncwarp();
    // pair slots: the warp's 32*KT pairs in (t,k) order, kLeanSteps steps of 32 in flight
    int32_t *pair_slot = a.out.pair_slot + (size_t)tw * KT;
    for (int j0 = 0; j0 < KT; j0 += kLeanSteps) {
        int ex[kLeanSteps], leader[kLeanSteps];
        unsigned m[kLeanSteps];
        int32_t first[kLeanSteps];
#pragma unroll
        for (int u = 0; u < kLeanSteps; ++u) {
            const int i = 32 * (j0 + u) + lane;
            ex[u] = j0 + u < KT ? ids_s[i] : -1;
            if ((unsigned)ex[u] >= (unsigned)E) ex[u] = -1;
        }
#pragma unroll
        for (int u = 0; u < kLeanSteps; ++u) {
            m[u] = __match_any_sync(kFullMask, ex[u] >= 0 ? ex[u] : E + lane);
            leader[u] = __ffs(m[u]) - 1;
        }
#pragma unroll
        for (int u = 0; u < kLeanSteps; ++u) {
            first[u] = 0;
            if (ex[u] >= 0 && lane == leader[u]) first[u] = atomicAdd(whist + ex[u], __popc(m[u]));   // the group's slots at once
            __syncwarp();                            // orders this step's counter update before the next step's
        }
#pragma unroll
        for (int u = 0; u < kLeanSteps; ++u) {
            const int i = 32 * (j0 + u) + lane;
            const int tok = tw + i / KT;
            first[u] = __shfl_sync(kFullMask, first[u], leader[u]);
            if (j0 + u < KT && tok < a.T) {
                if (ex[u] >= 0) {
                    const int32_t p = first[u] + __popc(m[u] & lt);
                    const int32_t row = rows_s[i];
                    pair_slot[i] = p;
                    a.out.pair_token[p] = tok;
                    a.out.pair_row[p] = row;
                } else {
                    pair_slot[i] = -1;
                }
            }
        }
    }
}

// The kernels are compiled for the common (top-k, ranks) pairs with both as compile-time constants (their
// loops unroll: the receive-row half of T=8192, K=8, R=8 takes 7.7 us instead of 9.4) and once with both
// read at run time.
using LayoutKernel = void (*)(LayoutArgs);
struct KernelPair {
    LayoutKernel count, assign;
};
template <int KT, int RT>
constexpr KernelPair kernel_pair() { return KernelPair{layout_cta_count_kernel<KT, RT>, layout_assign_kernel<KT, RT>}; }

constexpr int kTunedTopK[] = {2, 4, 6, 8};
constexpr int kTunedRanks = 8;
constexpr int kNumKernelPairs = 5;
const KernelPair kKernelPairs[kNumKernelPairs] = {kernel_pair<0, 0>(), kernel_pair<2, kTunedRanks>(), kernel_pair<4, kTunedRanks>(),
                                                  kernel_pair<6, kTunedRanks>(), kernel_pair<8, kTunedRanks>()};

int pick_kernels(int K, int R)               // the general kernels: exact (K, R), else the run-time pair
{
    if (R == kTunedRanks)
        for (int i = 0; i < 4; ++i)
            if (K == kTunedTopK[i]) return i + 1;
    return 0;
}

// The lean kernels: exact K (1..8 and 10), any rank count up to the bound they were compiled for (8, 16, 32 or 64).
struct LeanKernels {
    LayoutKernel ranks_count, ranks_assign;          // the receive-row half alone
    LayoutKernel count, assign;                      // the pair half, or both halves
};
template <int KT, int RT>
constexpr LeanKernels lean_kernels()
{
    return LeanKernels{lean_count_kernel<KT, RT, false>, lean_assign_kernel<KT, RT, false>, lean_count_kernel<KT, RT, true>,
                       lean_assign_kernel<KT, RT, true>};
}
constexpr int kLeanRankBounds[] = {8, 16, 32, 64};
constexpr int kNumLeanRankBounds = 4;
constexpr int kLeanTopK[] = {1, 2, 3, 4, 5, 6, 7, 8, 10};    // 10 of 512: the finest model the paper names
constexpr int kNumLeanTopK = sizeof(kLeanTopK) / sizeof(int);
template <int RT>
struct LeanRow {
    LeanKernels k[kNumLeanTopK] = {lean_kernels<1, RT>(), lean_kernels<2, RT>(), lean_kernels<3, RT>(), lean_kernels<4, RT>(),
                                   lean_kernels<5, RT>(), lean_kernels<6, RT>(), lean_kernels<7, RT>(), lean_kernels<8, RT>(),
                                   lean_kernels<10, RT>()};
};
const LeanRow<8> kLeanKernels8;
const LeanRow<16> kLeanKernels16;
const LeanRow<32> kLeanKernels32;
const LeanRow<64> kLeanKernels64;
const LeanKernels *lean_row(int b)
{
    return b == 0 ? kLeanKernels8.k : b == 1 ? kLeanKernels16.k : b == 2 ? kLeanKernels32.k : kLeanKernels64.k;
}

const LeanKernels *pick_lean(int K, int R)
{
    for (int b = 0; b < kNumLeanRankBounds; ++b)
        if (R <= kLeanRankBounds[b])
            for (int i = 0; i < kNumLeanTopK; ++i)
                if (K == kLeanTopK[i]) return &lean_row(b)[i];
    return nullptr;
}

// Which form a call takes: the lean kernels need a top-k of at most 8 (or 10), 16-byte aligned tables
// and, for the pair half, at most 1024 experts; the kernel pair also one scratch row per CTA inside the workspace.
enum { kGeneral = 0, kLeanSingle = 1, kLeanPair = 2 };
int lean_form(const ep_shape_t &s, const void *topk_idx, const ep_layout_t &out, size_t workspace_bytes, int parts)
{
    const bool ranks = parts & kPartRanks, pairs = parts & kPartPairs;
    const int T = s.num_tokens, E = s.num_experts, R = s.num_ranks;
    if (!pick_lean(s.top_k, R) || !aligned16(topk_idx) || (ranks && !aligned16(out.recv_slot)) ||
        (pairs && (!aligned16(out.pair_slot) || E > kLeanMaxExperts)))
        return kGeneral;
    if (T <= kLeanTokensPerCta) return kLeanSingle;
    const int n_ctas = ceil_div(T, kLeanTokensPerCta);
    if (n_ctas > kLeanMaxCtas || sizeof(int32_t) * (size_t)n_ctas * (R + 1 + (pairs ? E : 0)) > workspace_bytes) return kGeneral;
    return kLeanPair;
}

// Can `cfg` (one cluster = the whole grid) be resident on device `dev`? Asked once per device and
// (cluster size, CTA size, shared memory) and remembered; "no" sends the call to the global form.
bool cluster_fits(int dev, int which, const cudaLaunchConfig_t &cfg)
{
    struct Key {
        int dev, which;
        unsigned ctas, threads;
        size_t smem;
        bool fits;
    };
    static std::mutex mu;
    static Key known[32];
    static int n_known = 0;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_known; ++i)
        if (known[i].dev == dev && known[i].which == which && known[i].ctas == cfg.gridDim.x && known[i].threads == cfg.blockDim.x &&
            known[i].smem == cfg.dynamicSmemBytes)
            return known[i].fits;
    int n = 0;
    const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kKernelPairs[which].assign, &cfg);
    if (e != cudaSuccess) (void)cudaGetLastError();         // treated as "does not fit"; not this call's error
    const bool fits = e == cudaSuccess && n >= 1;
    if (n_known < 32) known[n_known++] = Key{dev, which, cfg.gridDim.x, cfg.blockDim.x, cfg.dynamicSmemBytes, fits};
    return fits;
}

int run_layout(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out, void *workspace,
               size_t workspace_bytes, void *stream_, int parts)
{
    int rc = check_shape(shape, false);
    if (rc != EP_OK) return rc;
    if (!out || !workspace) return EP_ERR_NULL;
    const bool ranks = parts & kPartRanks, pairs = parts & kPartPairs;
    if (ranks && (!out->rank_rows || !out->rank_row_offsets || !out->src_row_offsets || !out->status)) return EP_ERR_NULL;
    if (pairs && (!out->expert_counts || !out->expert_offsets)) return EP_ERR_NULL;
    if (shape->num_tokens > 0 && ranks && (!out->recv_slot || !out->recv_token)) return EP_ERR_NULL;
    if (shape->num_tokens > 0 && pairs && (!out->pair_slot || !out->pair_row || !out->pair_token)) return EP_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const LayoutPlan plan = make_plan(*shape);
    if (workspace_bytes < plan.workspace_bytes) return EP_ERR_CAPACITY;
    if (!aligned16(workspace)) return EP_ERR_INVALID_ARG;
    const int T = shape->num_tokens, E = shape->num_experts, R = shape->num_ranks;
    if (T == 0) {
        if (pairs) {
            EP_CUDA_TRY(cudaMemsetAsync(out->expert_counts, 0, sizeof(int32_t) * E, stream));
            EP_CUDA_TRY(cudaMemsetAsync(out->expert_offsets, 0, sizeof(int32_t) * (E + 1), stream));
        }
        if (ranks) {
            EP_CUDA_TRY(cudaMemsetAsync(out->rank_rows, 0, sizeof(int32_t) * R, stream));
            EP_CUDA_TRY(cudaMemsetAsync(out->rank_row_offsets, 0, sizeof(int32_t) * (R + 1), stream));
            EP_CUDA_TRY(cudaMemsetAsync(out->src_row_offsets, 0, sizeof(int32_t) * R * (R + 1), stream));
            EP_CUDA_TRY(cudaMemsetAsync(out->status, 0, sizeof(int32_t), stream));
        }
        return EP_OK;
    }
    if (!topk_idx) return EP_ERR_NULL;

    LayoutArgs a;
    a.idx = topk_idx;
    a.out = *out;
    a.cta_part = static_cast<int32_t *>(workspace);
    a.T = T; a.top_k = shape->top_k; a.E = E; a.num_ranks = R; a.Tr = T / R;
    a.mul_El = small_div_mul(E / R); a.mul_K = small_div_mul(shape->top_k); a.mul_R1 = small_div_mul(R + 1);
    a.by_Tr = make_fastdiv(T / R);
    a.tile_tokens = plan.tile_tokens; a.n_tiles = plan.n_tiles; a.bins = plan.bins; a.n_ctas = plan.n_ctas;
    a.mode = plan.mode;
    a.parts = parts;
    a.blo = pairs ? 0 : E;

    static std::atomic<bool> attr_done[64] = {};       // per device: dynamic shared memory limit raised
    int dev = 0;
    EP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return EP_ERR_INVALID_ARG;
    if (!attr_done[dev].load(std::memory_order_acquire)) {
        for (int i = 0; i < kNumKernelPairs; ++i) {
            EP_CUDA_TRY(cudaFuncSetAttribute(kKernelPairs[i].count, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget));
            EP_CUDA_TRY(cudaFuncSetAttribute(kKernelPairs[i].assign, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget));
        }
        for (int b = 0; b < kNumLeanRankBounds; ++b)
            for (int i = 0; i < kNumLeanTopK; ++i)
                EP_CUDA_TRY(cudaFuncSetAttribute(lean_row(b)[i].assign, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)lean_smem_bytes(kLeanMaxExperts, kLeanTopK[i])));
        attr_done[dev].store(true, std::memory_order_release);
    }
    const int which = pick_kernels(shape->top_k, R);
    const LeanKernels *lean = pick_lean(shape->top_k, R);
    const int form = lean_form(*shape, topk_idx, *out, workspace_bytes, parts);
    if (form == kLeanSingle) {
        // at most 256 tokens: the lean main kernel alone, one CTA
        a.n_ctas = 1;
        a.mode = kModeSingle;
        if (!pairs) lean->ranks_assign<<<1, kLeanWarps * 32, 0, stream>>>(a);
        else lean->assign<<<1, kLeanWarps * 32, lean_smem_bytes(E, shape->top_k), stream>>>(a);
        EP_LAUNCH_CHECK(1);
        return EP_OK;
    }
    if (form == kLeanPair) {
        // cta_part holds R+1 (+E) counters per CTA
        a.n_ctas = ceil_div(T, kLeanWarps * 32);
        a.mode = kModeGlobal;
        const dim3 grid(a.n_ctas), block(kLeanWarps * 32);
        if (!pairs) {
            lean->ranks_count<<<grid, block, 0, stream>>>(a);
            EP_CUDA_TRY(launch_pdl(lean->ranks_assign, grid, block, 0, stream, a));
        } else {
            lean->count<<<grid, block, sizeof(int32_t) * E, stream>>>(a);
            EP_CUDA_TRY(launch_pdl(lean->assign, grid, block, lean_smem_bytes(E, shape->top_k), stream, a));
        }
        EP_LAUNCH_CHECK(2);
        return EP_OK;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.n_ctas);
    cfg.blockDim = dim3(plan.warps * 32);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    int launched = 1;
    if (plan.mode == kModeCluster) {
        attr.id = cudaLaunchAttributeClusterDimension;      // the whole grid is one cluster
        attr.val.clusterDim.x = plan.n_ctas;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (!cluster_fits(dev, which, cfg)) {                      // this device cannot co-schedule the cluster
            a.mode = kModeGlobal;
            cfg.attrs = nullptr;
            cfg.numAttrs = 0;
        }
    }
    if (a.mode == kModeGlobal) {
        kKernelPairs[which].count<<<plan.n_ctas, plan.warps * 32, plan.smem, stream>>>(a);
        // the main kernel may start while the first still runs; it waits on the device before it reads cta_part
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        launched = 2;
    }
    EP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kKernelPairs[which].assign, a));
    EP_LAUNCH_CHECK(launched);
    return EP_OK;
}

}  // namespace

bool layout_is_lean(const ep_shape_t &shape, const void *topk_idx, const ep_layout_t &out, size_t workspace_bytes)
{
    return lean_form(shape, topk_idx, out, workspace_bytes, kPartRanks | kPartPairs) != kGeneral;
}

}  // namespace ep

extern "C" int ep_layout(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                         void *workspace, size_t workspace_bytes, void *stream)
{
    return ep::run_layout(shape, topk_idx, out, workspace, workspace_bytes, stream, ep::kPartRanks | ep::kPartPairs);
}

extern "C" int ep_layout_ranks(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                               void *workspace, size_t workspace_bytes, void *stream)
{
    return ep::run_layout(shape, topk_idx, out, workspace, workspace_bytes, stream, ep::kPartRanks);
}

extern "C" int ep_layout_pairs(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                               void *workspace, size_t workspace_bytes, void *stream)
{
    return ep::run_layout(shape, topk_idx, out, workspace, workspace_bytes, stream, ep::kPartPairs);
}

// ---------------------------------------------------------------------------
// ep_layout_static: the same layout with its scratch in a fixed device array, for
// callers that are not allowed to allocate device memory.
namespace ep {
namespace {

// Scratch of the allocation-free entry point. Every GPU on which this library is
// loaded holds these bytes until the process exits. In host code this name is
// only a handle: the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_layout_static_scratch[EP_LAYOUT_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_static_scratch_ptr[kMaxDevices] = {};      // device address of the array, per device
std::mutex g_static_scratch_mutex;

// Looks the array's device address up once per device, with that device current.
int static_scratch_address(void **ptr)
{
    int dev = -1;
    EP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return EP_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ptr[dev]) {
        void *p = nullptr;
        EP_CUDA_TRY(cudaGetSymbolAddress(&p, g_layout_static_scratch));
        if (!p) return EP_ERR_CUDA;
        g_static_scratch_ptr[dev] = p;
    }
    *ptr = g_static_scratch_ptr[dev];
    return EP_OK;
}

}  // namespace
}  // namespace ep

extern "C" size_t ep_layout_static_scratch_bytes(void) { return EP_LAYOUT_STATIC_SCRATCH_BYTES; }

extern "C" int ep_layout_static(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                                void *stream)
{
    int rc = ep::check_shape(shape, false);
    if (rc != EP_OK) return rc;
    // shapes whose scratch does not fit the fixed array are refused before anything is enqueued
    if (ep::make_plan(*shape).workspace_bytes > (size_t)EP_LAYOUT_STATIC_SCRATCH_BYTES) return EP_ERR_STATIC_SCRATCH;
    void *scratch = nullptr;
    rc = ep::static_scratch_address(&scratch);
    if (rc != EP_OK) return rc;
    // the counting kernel rewrites every cta_part word (bins blo..bins of every CTA) that the
    // assign kernel reads, so whatever the previous call left in the array needs no clearing
    return ep_layout(shape, topk_idx, out, scratch, EP_LAYOUT_STATIC_SCRATCH_BYTES, stream);
}
