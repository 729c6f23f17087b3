// Host-side entry points around the kernels: the copy-engine arm of the
// host-staged dispatch, the whole step from host buffers, the status read-back,
// bandwidth probes, and the error / launch bookkeeping.
#include <atomic>
#include <mutex>

#include "ep_common.cuh"

namespace ep {

namespace {
std::atomic<int> g_last_cuda_error{0};
std::atomic<long long> g_launches{0};
}  // namespace

// Timing-free events for cross-stream ordering: created on first use, kept for the life of the
// process (events hold no device memory). One pool per device, shared by every multi-stream entry
// point; `hold` keeps the pool's mutex until the caller has enqueued its whole sequence, so that
// two host threads cannot interleave their records and waits on the same events. (A wait that has
// been enqueued keeps the state the event had then; a later record by another call does not move it.)
namespace {
cudaEvent_t g_events[64][kOrderEventPool];
int g_events_ready[64] = {};
std::mutex g_event_mutex;
}  // namespace

int order_events(cudaEvent_t **pool, int need, std::unique_lock<std::mutex> &hold)
{
    if (need > kOrderEventPool) return EP_ERR_INVALID_ARG;
    int dev = 0;
    EP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return EP_ERR_INVALID_ARG;
    hold = std::unique_lock<std::mutex>(g_event_mutex);
    while (g_events_ready[dev] < need) {
        EP_CUDA_TRY(cudaEventCreateWithFlags(&g_events[dev][g_events_ready[dev]], cudaEventDisableTiming));
        ++g_events_ready[dev];
    }
    *pool = g_events[dev];
    return EP_OK;
}

void note_cuda_error(cudaError_t e) { g_last_cuda_error.store((int)e); }
void count_launches(int n) { g_launches.fetch_add(n); }

namespace {

// ---- probes: 16-byte streams, one small CTA per 16 KB chunk (256 threads x 4 vectors). Measured on
// B200, this shape gives the highest figures (writes 7.0-7.3 TB/s against 6.0-6.5 TB/s from a
// persistent grid-stride loop), and it is the shape of the row movers.
constexpr int kProbeThreads = 256, kProbeVecs = 4;

__global__ void probe_read_kernel(const uint4 *src, size_t n_vec, uint4 *sink)
{
    uint4 acc = make_uint4(0, 0, 0, 0);
    const size_t base = (size_t)blockIdx.x * kProbeThreads * kProbeVecs + threadIdx.x;
    uint4 v[kProbeVecs];
#pragma unroll
    for (int u = 0; u < kProbeVecs; ++u)
        if (base + (size_t)u * kProbeThreads < n_vec) v[u] = ld_stream(src + base + (size_t)u * kProbeThreads);
        else v[u] = acc;
#pragma unroll
    for (int u = 0; u < kProbeVecs; ++u) {
        acc.x ^= v[u].x; acc.y ^= v[u].y; acc.z ^= v[u].z; acc.w ^= v[u].w;
    }
    if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x9e3779b9u) *sink = acc;   // keeps the loads alive, practically never taken
}

__global__ void probe_write_kernel(uint4 *dst, size_t n_vec)
{
    const uint4 v = make_uint4(threadIdx.x, blockIdx.x, 0x3f803f80u, 0x3f803f80u);
    const size_t base = (size_t)blockIdx.x * kProbeThreads * kProbeVecs + threadIdx.x;
#pragma unroll
    for (int u = 0; u < kProbeVecs; ++u)
        if (base + (size_t)u * kProbeThreads < n_vec) st_stream(dst + base + (size_t)u * kProbeThreads, v);
}

__global__ void probe_copy_kernel(uint4 *dst, const uint4 *src, size_t n_vec)
{
    const size_t base = (size_t)blockIdx.x * kProbeThreads * kProbeVecs + threadIdx.x;
    uint4 v[kProbeVecs];
#pragma unroll
    for (int u = 0; u < kProbeVecs; ++u)
        if (base + (size_t)u * kProbeThreads < n_vec) v[u] = ld_stream(src + base + (size_t)u * kProbeThreads);
#pragma unroll
    for (int u = 0; u < kProbeVecs; ++u)
        if (base + (size_t)u * kProbeThreads < n_vec) st_stream(dst + base + (size_t)u * kProbeThreads, v[u]);
}

struct Carver {
    char *p;
    size_t used = 0;
    explicit Carver(void *base) : p(static_cast<char *>(base)) {}
    template <class T>
    T *take(size_t count)
    {
        T *r = reinterpret_cast<T *>(p ? p + used : nullptr);
        used += (count * sizeof(T) + 255) & ~size_t(255);
        return r;
    }
};

struct StepBuffers {
    uint16_t *x, *recv, *grouped, *y;
    int32_t *idx;
    float *w;
    ep_layout_t lay;
    void *workspace;
    size_t workspace_bytes;
    int64_t recv_rows, pair_rows;
    size_t total;
};

// `half` picks one of the two copies of what the copy streams touch (x, topk_idx, topk_weights, y and the
// status word), so that a step's uploads and downloads need not wait for the step before it; everything else
// is used on the compute stream only and is ordered by it.
StepBuffers carve_step(const ep_shape_t &s, void *arena, int half = 0)
{
    StepBuffers b;
    const size_t T = s.num_tokens, K = s.top_k, H = s.hidden, E = s.num_experts, R = s.num_ranks;
    const size_t TK = T * K, rows = T * (K < R ? K : R);
    Carver c(arena);
    b.recv_rows = (int64_t)rows;
    b.pair_rows = (int64_t)TK;
    for (int h = 0; h < 2; ++h) {
        uint16_t *x = c.take<uint16_t>(T * H), *y = c.take<uint16_t>(T * H);
        int32_t *idx = c.take<int32_t>(TK);
        float *w = c.take<float>(TK);
        int32_t *status = c.take<int32_t>(1);
        if (h == half) {
            b.x = x; b.y = y; b.idx = idx; b.w = w; b.lay.status = status;
        }
    }
    b.recv = c.take<uint16_t>(rows * H);
    b.grouped = c.take<uint16_t>(TK * H);
    b.lay.expert_counts = c.take<int32_t>(E);
    b.lay.expert_offsets = c.take<int32_t>(E + 1);
    b.lay.rank_rows = c.take<int32_t>(R);
    b.lay.rank_row_offsets = c.take<int32_t>(R + 1);
    b.lay.src_row_offsets = c.take<int32_t>(R * (R + 1));
    b.lay.recv_slot = c.take<int32_t>(TK);
    b.lay.pair_slot = c.take<int32_t>(TK);
    b.lay.recv_token = c.take<int32_t>(rows);
    b.lay.pair_row = c.take<int32_t>(TK);
    b.lay.pair_token = c.take<int32_t>(TK);
    b.workspace_bytes = ep_layout_workspace_bytes(&s);
    b.workspace = c.take<char>(b.workspace_bytes);
    b.total = c.used;
    return b;
}

}  // namespace
}  // namespace ep

extern "C" int ep_dispatch_copy_engine(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                                       const int32_t *rank_row_offsets_host, void *staging,
                                       int64_t staging_capacity_rows, void *recv_host, int32_t *status,
                                       void *stream_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x || !recv_slot || !staging || !recv_host) return EP_ERR_NULL;
    if (!aligned16(x) || !aligned16(staging) || staging_capacity_rows < 0) return EP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t row_bytes = (size_t)shape->hidden * 2;
    if (rank_row_offsets_host) {
        const int R = shape->num_ranks;
        if (rank_row_offsets_host[0] != 0 || rank_row_offsets_host[R] > staging_capacity_rows) return EP_ERR_CAPACITY;
        for (int r = 0; r < R; ++r)
            if (rank_row_offsets_host[r + 1] < rank_row_offsets_host[r]) return EP_ERR_INVALID_ARG;
    }
    rc = launch_dispatch(*shape, x, recv_slot, staging, staging_capacity_rows, status, stream);
    if (rc != EP_OK) return rc;
    if (rank_row_offsets_host) {
        for (int r = 0; r < shape->num_ranks; ++r) {          // one contiguous region per destination rank
            const size_t lo = (size_t)rank_row_offsets_host[r], hi = (size_t)rank_row_offsets_host[r + 1];
            if (hi > lo)
                EP_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(recv_host) + lo * row_bytes,
                                            static_cast<const char *>(staging) + lo * row_bytes,
                                            (hi - lo) * row_bytes, cudaMemcpyDeviceToHost, stream));
        }
    } else if (staging_capacity_rows > 0) {
        EP_CUDA_TRY(cudaMemcpyAsync(recv_host, staging, (size_t)staging_capacity_rows * row_bytes,
                                    cudaMemcpyDeviceToHost, stream));
    }
    return EP_OK;
}

extern "C" size_t ep_host_step_arena_bytes(const ep_shape_t *shape)
{
    if (ep::check_shape(shape, true) != EP_OK) return 0;
    return ep::carve_step(*shape, nullptr).total;
}

extern "C" int ep_host_step(const ep_shape_t *shape, const void *x_host, const int32_t *topk_idx_host,
                            const float *topk_weights_host, void *y_host, int32_t *status_host, void *arena,
                            size_t arena_bytes, void *stream_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (!arena) return EP_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return EP_ERR_INVALID_ARG;
    const StepBuffers b = carve_step(*shape, arena);
    if (arena_bytes < b.total) return EP_ERR_CAPACITY;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x_host || !topk_idx_host || !topk_weights_host || !y_host) return EP_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t T = shape->num_tokens, K = shape->top_k, H = shape->hidden;
    EP_CUDA_TRY(cudaMemcpyAsync(b.idx, topk_idx_host, T * K * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    EP_CUDA_TRY(cudaMemcpyAsync(b.w, topk_weights_host, T * K * sizeof(float), cudaMemcpyHostToDevice, stream));
    EP_CUDA_TRY(cudaMemcpyAsync(b.x, x_host, T * H * 2, cudaMemcpyHostToDevice, stream));
    rc = ep_layout(shape, b.idx, &b.lay, b.workspace, b.workspace_bytes, stream);
    if (rc != EP_OK) return rc;
    rc = launch_dispatch(*shape, b.x, b.lay.recv_slot, b.recv, b.recv_rows, b.lay.status, stream);
    if (rc != EP_OK) return rc;
    rc = launch_group(*shape, b.recv, b.recv_rows, b.lay.pair_row, b.lay.expert_offsets + shape->num_experts,
                      b.grouped, b.pair_rows, b.lay.status, stream);
    if (rc != EP_OK) return rc;
    rc = launch_combine(*shape, b.grouped, b.pair_rows, b.lay.pair_slot, b.w, b.y, b.lay.status, stream);
    if (rc != EP_OK) return rc;
    EP_CUDA_TRY(cudaMemcpyAsync(y_host, b.y, T * H * 2, cudaMemcpyDeviceToHost, stream));
    if (status_host)
        EP_CUDA_TRY(cudaMemcpyAsync(status_host, b.lay.status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    return EP_OK;
}

extern "C" int ep_host_step_pipelined(const ep_shape_t *shape, const void *x_host, const int32_t *topk_idx_host,
                                      const float *topk_weights_host, void *y_host, int32_t *status_host,
                                      void *arena, size_t arena_bytes, int chunks, void *stream_in_,
                                      void *stream_compute_, void *stream_out_, int round, void *const *step_events)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (!arena) return EP_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0 || chunks < 1 || chunks > 256 || round < 0) return EP_ERR_INVALID_ARG;
    if (step_events && (!step_events[0] || !step_events[1] || !step_events[2] || !step_events[3])) return EP_ERR_NULL;
    const int half = step_events ? (round & 1) : 0;
    const StepBuffers b = carve_step(*shape, arena, half);
    if (arena_bytes < b.total) return EP_ERR_CAPACITY;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x_host || !topk_idx_host || !topk_weights_host || !y_host) return EP_ERR_NULL;
    cudaStream_t in = static_cast<cudaStream_t>(stream_in_), comp = static_cast<cudaStream_t>(stream_compute_),
                 outs = static_cast<cudaStream_t>(stream_out_);
    cudaEvent_t *ev = nullptr;
    std::unique_lock<std::mutex> hold;
    rc = order_events(&ev, 2 * chunks + 3, hold);
    if (rc != EP_OK) return rc;
    const size_t T = shape->num_tokens, K = shape->top_k, H = shape->hidden;
    if (step_events) {
        // this half of the arena was last used two steps ago: its uploads wait for that step's kernels and its
        // kernels for that step's downloads, not for the step before this one, whose transfers are still running
        EP_CUDA_TRY(cudaStreamWaitEvent(in, static_cast<cudaEvent_t>(step_events[half]), 0));
        EP_CUDA_TRY(cudaStreamWaitEvent(comp, static_cast<cudaEvent_t>(step_events[2 + half]), 0));
    } else {
        // one half, reused from step to step: uploads wait for the previous step's kernels, and the kernels
        // for the previous step's downloads of y
        EP_CUDA_TRY(cudaEventRecord(ev[0], comp));
        EP_CUDA_TRY(cudaStreamWaitEvent(in, ev[0], 0));
        EP_CUDA_TRY(cudaEventRecord(ev[1], outs));
        EP_CUDA_TRY(cudaStreamWaitEvent(comp, ev[1], 0));
    }
    EP_CUDA_TRY(cudaMemcpyAsync(b.idx, topk_idx_host, T * K * sizeof(int32_t), cudaMemcpyHostToDevice, in));
    EP_CUDA_TRY(cudaMemcpyAsync(b.w, topk_weights_host, T * K * sizeof(float), cudaMemcpyHostToDevice, in));
    EP_CUDA_TRY(cudaEventRecord(ev[2], in));
    EP_CUDA_TRY(cudaStreamWaitEvent(comp, ev[2], 0));
    rc = ep_layout(shape, b.idx, &b.lay, b.workspace, b.workspace_bytes, comp);
    if (rc != EP_OK) return rc;
    for (int c = 0; c < chunks; ++c) {
        const size_t t0 = T * c / chunks, t1 = T * (c + 1) / chunks, n = t1 - t0;
        if (n == 0) continue;
        ep_shape_t part = *shape;
        part.num_tokens = (int32_t)n;
        // upload this chunk of x while earlier chunks are being processed and downloaded
        EP_CUDA_TRY(cudaMemcpyAsync(b.x + t0 * H, static_cast<const uint16_t *>(x_host) + t0 * H, n * H * 2,
                                    cudaMemcpyHostToDevice, in));
        EP_CUDA_TRY(cudaEventRecord(ev[3 + 2 * c], in));
        EP_CUDA_TRY(cudaStreamWaitEvent(comp, ev[3 + 2 * c], 0));
        rc = launch_dispatch(part, b.x + t0 * H, b.lay.recv_slot + t0 * K, b.recv, b.recv_rows, b.lay.status, comp);
        if (rc != EP_OK) return rc;
        // identity expert: the chunk's pair rows are its receive rows
        rc = launch_permute(shape->hidden, b.recv, b.recv_rows, b.lay.recv_slot + t0 * K, b.grouped, b.pair_rows,
                            b.lay.pair_slot + t0 * K, (int64_t)(n * K), b.lay.status, comp);
        if (rc != EP_OK) return rc;
        rc = launch_combine(part, b.grouped, b.pair_rows, b.lay.pair_slot + t0 * K, b.w + t0 * K, b.y + t0 * H,
                            b.lay.status, comp);
        if (rc != EP_OK) return rc;
        EP_CUDA_TRY(cudaEventRecord(ev[4 + 2 * c], comp));
        EP_CUDA_TRY(cudaStreamWaitEvent(outs, ev[4 + 2 * c], 0));
        EP_CUDA_TRY(cudaMemcpyAsync(static_cast<uint16_t *>(y_host) + t0 * H, b.y + t0 * H, n * H * 2,
                                    cudaMemcpyDeviceToHost, outs));
    }
    if (status_host)
        EP_CUDA_TRY(cudaMemcpyAsync(status_host, b.lay.status, sizeof(int32_t), cudaMemcpyDeviceToHost, outs));
    if (step_events) {
        EP_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(step_events[half]), comp));
        EP_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(step_events[2 + half]), outs));
    }
    return EP_OK;
}

extern "C" int ep_status(const int32_t *status_dev, void *stream_, int32_t *status_host)
{
    if (!status_dev || !status_host) return EP_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    EP_CUDA_TRY(cudaMemcpyAsync(status_host, status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    EP_CUDA_TRY(cudaStreamSynchronize(stream));
    return EP_OK;
}

extern "C" int ep_probe_bandwidth(int kind, void *dst, const void *src, size_t bytes, int iters, void *stream_,
                                  double *gbs)
{
    using namespace ep;
    if (!gbs) return EP_ERR_NULL;
    if (kind < EP_PROBE_READ || kind > EP_PROBE_MEMCPY || bytes == 0 || bytes % 16 != 0 || iters < 1)
        return EP_ERR_INVALID_ARG;
    const bool need_src = kind != EP_PROBE_WRITE, need_dst = true;   // the read probe needs a 16-byte sink
    if ((need_src && !src) || (need_dst && !dst)) return EP_ERR_NULL;
    if (kind != EP_PROBE_MEMCPY && ((need_src && !aligned16(src)) || !aligned16(dst))) return EP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int dev = 0, sms = 0;
    EP_CUDA_TRY(cudaGetDevice(&dev));
    EP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cudaEvent_t e0, e1;
    EP_CUDA_TRY(cudaEventCreate(&e0));
    cudaError_t ce = cudaEventCreate(&e1);
    if (ce != cudaSuccess) {
        cudaEventDestroy(e0);
        note_cuda_error(ce);
        return EP_ERR_CUDA;
    }
    const size_t n_vec = bytes / 16;
    const int block = kProbeThreads;
    const unsigned grid = (unsigned)((n_vec + (size_t)kProbeThreads * kProbeVecs - 1) / ((size_t)kProbeThreads * kProbeVecs));
    (void)sms;
    float best_ms = 1e30f;
    int rc = EP_OK;
    for (int it = 0; it < iters + 1 && rc == EP_OK; ++it) {       // first repetition is a warm-up
        cudaEventRecord(e0, stream);
        switch (kind) {
        case EP_PROBE_READ:
            probe_read_kernel<<<grid, block, 0, stream>>>(static_cast<const uint4 *>(src), n_vec, static_cast<uint4 *>(dst));
            count_launches(1);
            break;
        case EP_PROBE_WRITE:
            probe_write_kernel<<<grid, block, 0, stream>>>(static_cast<uint4 *>(dst), n_vec);
            count_launches(1);
            break;
        case EP_PROBE_COPY:
            probe_copy_kernel<<<grid, block, 0, stream>>>(static_cast<uint4 *>(dst), static_cast<const uint4 *>(src), n_vec);
            count_launches(1);
            break;
        default: {
            cudaError_t e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, stream);
            if (e != cudaSuccess) { note_cuda_error(e); rc = EP_ERR_CUDA; }
        }
        }
        cudaEventRecord(e1, stream);
        cudaError_t e = cudaEventSynchronize(e1);
        if (e != cudaSuccess) { note_cuda_error(e); rc = EP_ERR_CUDA; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (it > 0 && ms < best_ms) best_ms = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != EP_OK) return rc;
    const double moved = (kind == EP_PROBE_COPY ? 2.0 : 1.0) * (double)bytes;
    *gbs = moved / (best_ms * 1e-3) / 1e9;
    return EP_OK;
}

extern "C" int64_t ep_launch_count(void) { return ep::g_launches.load(); }

extern "C" const char *ep_strerror(int err)
{
    switch (err) {
    case EP_OK: return "ok";
    case EP_ERR_NULL: return "a required pointer is NULL";
    case EP_ERR_INVALID_ARG: return "invalid argument (shape outside the supported limits or misaligned buffer)";
    case EP_ERR_CAPACITY: return "a caller-provided buffer is too small";
    case EP_ERR_CUDA: return "a CUDA runtime call failed (see ep_last_cuda_error)";
    case EP_ERR_STATIC_SCRATCH:
        return "ep_layout_static: this shape needs more scratch than the library's fixed array holds; "
               "use ep_layout with a caller-provided workspace";
    default: return "unknown error";
    }
}

extern "C" int ep_last_cuda_error(void) { return ep::g_last_cuda_error.load(); }
