// ep_layout: counts, prefix scans and deterministic destination slots, all on the device.
//
// The work is a stable counting sort of the T*K (token, k) pairs by expert id plus
// a stable count of the distinct (token, rank) hits. Determinism never depends on
// the arrival order of atomics: tokens are cut into contiguous tiles, one warp
// owns a tile, and every rank inside a tile is derived from warp ballots /
// matches whose lane order is the (t,k) order.
//
//   pass 1  count   one warp per tile: histogram of experts, of rank hits and of
//                   bad ids over the tile            -> part[tile][bin]
//   pass 2  scan    one warp per bin: exclusive scan of part[.][bin] over tiles
//                   (in place) and the bin total; the last CTA to finish scans
//                   the totals over bins             -> counts, offsets, status
//   pass 3  assign  one warp per tile: replays the tile in order with running
//                   counters that start at offset[bin] + part[tile][bin]
//                                                    -> slots and inverse maps
//
// Bins: [0,E) experts, [E,E+R) rank hits, [E+R] ids outside [-1,E).
#include <mutex>

#include "ep_common.cuh"

namespace ep {
namespace {

constexpr int kMaxTiles = 1024;     // lanes of the scan warp own <= 32 tiles each
constexpr int kScanWarps = 4;

struct LayoutPlan {
    int tile_tokens;    // tokens per tile, a multiple of 32
    int n_tiles;
    int bins;           // E + R + 1
    int warps;          // warps (tiles) per CTA in pass 1 and 3
    size_t smem_count;  // dynamic shared memory, pass 1
    size_t smem_assign; // dynamic shared memory, pass 3
    size_t workspace_bytes;
};

LayoutPlan make_plan(const ep_shape_t &s)
{
    LayoutPlan p;
    const int T = s.num_tokens;
    int per = ceil_div(ceil_div(T > 0 ? T : 1, kMaxTiles), 32) * 32;
    p.tile_tokens = per < 32 ? 32 : per;
    p.n_tiles = ceil_div(T, p.tile_tokens);
    p.bins = s.num_experts + s.num_ranks + 1;
    // per-warp shared memory of pass 3: running counters + ballots + staged receive slots
    size_t per_warp = sizeof(int32_t) * (size_t)(p.bins + kMaxRanks + 32 * s.top_k);
    int w = (int)((96 * 1024) / per_warp);
    p.warps = w < 1 ? 1 : (w > 8 ? 8 : w);
    p.smem_assign = per_warp * p.warps;
    p.smem_count = sizeof(int32_t) * (size_t)p.bins * p.warps;
    p.workspace_bytes = sizeof(int32_t) * ((size_t)(p.n_tiles > 0 ? p.n_tiles : 1) * p.bins + p.bins + 4);
    return p;
}

struct LayoutArgs {
    const int32_t *idx;
    ep_layout_t out;
    int32_t *part;      // [n_tiles][bins]
    int32_t *totals;    // [bins]
    unsigned *ticket;   // [1]
    int T, K, E, R, El, Tr;
    int tile_tokens, n_tiles, bins;
};

// ---------------------------------------------------------------- pass 1
__global__ void layout_count_kernel(LayoutArgs a)
{
    extern __shared__ int32_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x * (blockDim.x >> 5) + warp;
    if (blockIdx.x == 0 && threadIdx.x == 0) *a.ticket = 0u;     // pass 2 counts finished CTAs here
    if (tile >= a.n_tiles) return;
    int32_t *hist = smem + warp * a.bins;
    for (int b = lane; b < a.bins; b += 32) hist[b] = 0;
    __syncwarp();

    const int t0 = tile * a.tile_tokens;
    const int t1 = min(a.T, t0 + a.tile_tokens);
    // experts: any order
    int bad = 0;
    for (int i = t0 * a.K + lane; i < t1 * a.K; i += 32) {
        const int e = __ldg(a.idx + i);
        if (e >= 0 && e < a.E) atomicAdd(hist + e, 1);
        else if (e != -1) ++bad;
    }
    if (bad) atomicAdd(hist + a.E + a.R, bad);
    // rank hits: one token per lane, one ballot per rank
    for (int tb = t0; tb < t1; tb += 32) {
        const int t = tb + lane;
        unsigned long long mask = 0ull;
        if (t < t1)
            for (int k = 0; k < a.K; ++k) {
                const int e = __ldg(a.idx + (size_t)t * a.K + k);
                if (e >= 0 && e < a.E) mask |= 1ull << (e / a.El);
            }
        for (int r = 0; r < a.R; ++r) {
            const unsigned b = __ballot_sync(kFullMask, (mask >> r) & 1ull);
            if (lane == 0) hist[a.E + r] += __popc(b);
        }
    }
    __syncwarp();
    int32_t *dst = a.part + (size_t)tile * a.bins;
    for (int b = lane; b < a.bins; b += 32) dst[b] = hist[b];
}

// ---------------------------------------------------------------- pass 2
// exclusive scan of in[0..n) into out[0..n], out[n] = total; whole CTA, n <= 4096+
__device__ void block_exclusive_scan(const int32_t *in, int32_t *out, int n, int32_t *sh /* [blockDim.x] */)
{
    const int nt = blockDim.x, tid = threadIdx.x;
    const int chunk = (n + nt - 1) / nt;
    const int lo = min(n, tid * chunk), hi = min(n, lo + chunk);
    int32_t sum = 0;
    for (int i = lo; i < hi; ++i) sum += __ldcg(in + i);     // written by other CTAs: read at L2
    sh[tid] = sum;
    __syncthreads();
    for (int off = 1; off < nt; off <<= 1) {      // Hillis-Steele inclusive scan over the chunk sums
        int32_t v = tid >= off ? sh[tid - off] : 0;
        __syncthreads();
        sh[tid] += v;
        __syncthreads();
    }
    int32_t run = sh[tid] - sum;
    for (int i = lo; i < hi; ++i) {
        const int32_t v = __ldcg(in + i);
        out[i] = run;
        run += v;
    }
    if (tid == nt - 1) out[n] = sh[tid];
    __syncthreads();
}

__global__ void layout_scan_kernel(LayoutArgs a)
{
    __shared__ int32_t sh[kScanWarps * 32];
    __shared__ bool is_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bin = blockIdx.x * kScanWarps + warp;
    if (bin < a.bins) {
        const int c = (a.n_tiles + 31) >> 5;                   // tiles owned by a lane, contiguous
        const int lo = min(a.n_tiles, lane * c), hi = min(a.n_tiles, lo + c);
        int32_t sum = 0;
        for (int j = lo; j < hi; ++j) sum += a.part[(size_t)j * a.bins + bin];
        int32_t incl = sum;
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t v = __shfl_up_sync(kFullMask, incl, off);
            if (lane >= off) incl += v;
        }
        int32_t run = incl - sum;
        for (int j = lo; j < hi; ++j) {
            int32_t *p = a.part + (size_t)j * a.bins + bin;
            const int32_t v = *p;
            *p = run;
            run += v;
        }
        if (lane == 31) {
            a.totals[bin] = incl;
            if (bin < a.E) a.out.expert_counts[bin] = incl;
            else if (bin < a.E + a.R) a.out.rank_rows[bin - a.E] = incl;
        }
    }
    // the last CTA to get here scans the totals over the bins
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(a.ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    block_exclusive_scan(a.totals, a.out.expert_offsets, a.E, sh);
    block_exclusive_scan(a.totals + a.E, a.out.rank_row_offsets, a.R, sh);
    for (int r = threadIdx.x; r < a.R; r += blockDim.x)
        a.out.src_row_offsets[r * (a.R + 1) + a.R] = a.out.rank_row_offsets[r + 1];
    if (threadIdx.x == 0) *a.out.status = __ldcg(a.totals + a.E + a.R) ? EP_STATUS_BAD_INDEX : 0;
}

// ---------------------------------------------------------------- pass 3
__global__ void layout_assign_kernel(LayoutArgs a)
{
    extern __shared__ int32_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x * (blockDim.x >> 5) + warp;
    if (tile >= a.n_tiles) return;
    const int nb = a.E + a.R;
    const int per_warp = a.bins + kMaxRanks + 32 * a.K;
    int32_t *run = smem + warp * per_warp;           // [E+R] next free slot of each bin
    unsigned *bal = reinterpret_cast<unsigned *>(run + a.bins);   // [R] ballot of the current 32 tokens
    int32_t *slot_s = run + a.bins + kMaxRanks;      // [32*K] receive slots of the current 32 tokens
    const unsigned lt = lanemask_lt();

    const int32_t *base = a.part + (size_t)tile * a.bins;
    for (int b = lane; b < nb; b += 32)
        run[b] = base[b] + (b < a.E ? a.out.expert_offsets[b] : a.out.rank_row_offsets[b - a.E]);
    __syncwarp();

    const int t0 = tile * a.tile_tokens;
    const int t1 = min(a.T, t0 + a.tile_tokens);
    for (int tb = t0; tb < t1; tb += 32) {
        const int t = tb + lane;
        const bool live = t < t1;
        // --- receive rows: which of these 32 tokens hit which rank
        unsigned long long mask = 0ull;
        if (live)
            for (int k = 0; k < a.K; ++k) {
                const int e = __ldg(a.idx + (size_t)t * a.K + k);
                if (e >= 0 && e < a.E) mask |= 1ull << (e / a.El);
            }
        for (int r = 0; r < a.R; ++r) {
            const unsigned b = __ballot_sync(kFullMask, (mask >> r) & 1ull);
            if (lane == 0) bal[r] = b;
        }
        __syncwarp();
        if (live) {
            if (t % a.Tr == 0) {                     // first token of a source rank
                const int s = t / a.Tr;
                for (int r = 0; r < a.R; ++r)
                    a.out.src_row_offsets[r * (a.R + 1) + s] = run[a.E + r] + __popc(bal[r] & lt);
            }
            unsigned long long seen = 0ull;
            for (int k = 0; k < a.K; ++k) {
                const int e = __ldg(a.idx + (size_t)t * a.K + k);
                int32_t row = -1;
                if (e >= 0 && e < a.E) {
                    const int r = e / a.El;
                    row = run[a.E + r] + __popc(bal[r] & lt);
                    if (!((seen >> r) & 1ull)) {
                        a.out.recv_token[row] = t;
                        seen |= 1ull << r;
                    }
                }
                slot_s[lane * a.K + k] = row;
            }
        }
        __syncwarp();
        for (int r = lane; r < a.R; r += 32) run[a.E + r] += __popc(bal[r]);
        __syncwarp();
        // --- pair slots: the items of these tokens, 32 at a time in (t,k) order
        const int n_items = (min(t1, tb + 32) - tb) * a.K;
        const size_t i0 = (size_t)tb * a.K;
        for (int j = 0; j < n_items; j += 32) {
            const int i = j + lane;
            const bool act = i < n_items;
            const int e = act ? __ldg(a.idx + i0 + i) : -1;
            const bool valid = act && e >= 0 && e < a.E;
            const unsigned m = __match_any_sync(kFullMask, valid ? e : a.E + lane);
            int32_t first = 0;
            if (valid) {
                first = run[e];
                const int32_t p = first + __popc(m & lt);
                const int32_t row = slot_s[i];
                a.out.pair_slot[i0 + i] = p;
                a.out.recv_slot[i0 + i] = row;
                a.out.pair_token[p] = tb + i / a.K;
                a.out.pair_row[p] = row;
            } else if (act) {
                a.out.pair_slot[i0 + i] = -1;
                a.out.recv_slot[i0 + i] = -1;
            }
            __syncwarp();
            if (valid && (m >> lane) <= 1u) run[e] = first + __popc(m);   // highest lane of the group
            __syncwarp();
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

extern "C" int ep_layout(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                         void *workspace, size_t workspace_bytes, void *stream_)
{
    using namespace ep;
    int rc = check_shape(shape, false);
    if (rc != EP_OK) return rc;
    if (!out || !workspace) return EP_ERR_NULL;
    if (!out->expert_counts || !out->expert_offsets || !out->rank_rows || !out->rank_row_offsets ||
        !out->src_row_offsets || !out->status)
        return EP_ERR_NULL;
    if (shape->num_tokens > 0 && (!out->recv_slot || !out->pair_slot || !out->recv_token || !out->pair_row ||
                                  !out->pair_token))
        return EP_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const LayoutPlan plan = make_plan(*shape);
    if (workspace_bytes < plan.workspace_bytes) return EP_ERR_CAPACITY;
    if (!aligned16(workspace)) return EP_ERR_INVALID_ARG;
    const int T = shape->num_tokens, E = shape->num_experts, R = shape->num_ranks;
    if (T == 0) {
        EP_CUDA_TRY(cudaMemsetAsync(out->expert_counts, 0, sizeof(int32_t) * E, stream));
        EP_CUDA_TRY(cudaMemsetAsync(out->expert_offsets, 0, sizeof(int32_t) * (E + 1), stream));
        EP_CUDA_TRY(cudaMemsetAsync(out->rank_rows, 0, sizeof(int32_t) * R, stream));
        EP_CUDA_TRY(cudaMemsetAsync(out->rank_row_offsets, 0, sizeof(int32_t) * (R + 1), stream));
        EP_CUDA_TRY(cudaMemsetAsync(out->src_row_offsets, 0, sizeof(int32_t) * R * (R + 1), stream));
        EP_CUDA_TRY(cudaMemsetAsync(out->status, 0, sizeof(int32_t), stream));
        return EP_OK;
    }
    if (!topk_idx) return EP_ERR_NULL;

    LayoutArgs a;
    a.idx = topk_idx;
    a.out = *out;
    a.part = static_cast<int32_t *>(workspace);
    a.totals = a.part + (size_t)plan.n_tiles * plan.bins;
    a.ticket = reinterpret_cast<unsigned *>(a.totals + plan.bins);
    a.T = T; a.K = shape->top_k; a.E = E; a.R = R; a.El = E / R; a.Tr = T / R;
    a.tile_tokens = plan.tile_tokens; a.n_tiles = plan.n_tiles; a.bins = plan.bins;

    static bool attr_done[64] = {};
    int dev = 0;
    EP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 64 && !attr_done[dev]) {
        EP_CUDA_TRY(cudaFuncSetAttribute(layout_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
        EP_CUDA_TRY(cudaFuncSetAttribute(layout_assign_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
        attr_done[dev] = true;
    }
    const int grid_tiles = ceil_div(plan.n_tiles, plan.warps);
    layout_count_kernel<<<grid_tiles, plan.warps * 32, plan.smem_count, stream>>>(a);
    layout_scan_kernel<<<ceil_div(plan.bins, kScanWarps), kScanWarps * 32, 0, stream>>>(a);
    layout_assign_kernel<<<grid_tiles, plan.warps * 32, plan.smem_assign, stream>>>(a);
    EP_LAUNCH_CHECK(3);
    return EP_OK;
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
    // pass 1 rewrites every scratch word it later reads (including the CTA ticket),
    // so whatever the previous call left in the array needs no clearing
    return ep_layout(shape, topk_idx, out, scratch, EP_LAYOUT_STATIC_SCRATCH_BYTES, stream);
}
