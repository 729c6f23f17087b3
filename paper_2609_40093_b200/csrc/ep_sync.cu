// Per-sender completion flags with bounded polling, and the host-staged round trip
// that uses separate upload / download streams.
//
// Flags live apart from the payload (one 32-bit word per sender, single writer, no
// atomics). The wait kernel gives one thread to each sender: it polls the sender's
// flag with volatile system-scope loads and sleeps between attempts; when the flag
// carries the expected epoch the thread publishes the epoch in a device-memory word
// that consumer threads can watch cheaply. Every wait is bounded twice (wall time
// on %globaltimer and an iteration count): when the bound is hit the thread gives
// up, sets EP_STATUS_TIMEOUT and the kernel returns, so the stream and the context
// stay usable.
#include "ep_common.cuh"

namespace ep {


namespace {

constexpr unsigned long long kMaxTimeoutNs = 2000000000ull;   // 2 s
constexpr int kMaxSenders = 64;

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ uint32_t load_flag(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void wait_senders_kernel(const uint32_t *flags, int n, uint32_t epoch, unsigned long long timeout_ns,
                                    uint32_t *arrived, int32_t *status)
{
    const int s = threadIdx.x;
    if (s >= n) return;
    const unsigned long long t0 = global_timer_ns();
    const unsigned long long max_iters = timeout_ns / 64 + 1024;     // second bound, should the timer misbehave
    bool ok = false;
    unsigned pause_ns = 32;
    for (unsigned long long it = 0; it < max_iters; ++it) {
        if (load_flag(flags + s) == epoch) {
            ok = true;
            break;
        }
        if (global_timer_ns() - t0 > timeout_ns) break;
        __nanosleep(pause_ns);                                        // pause between attempts
        if (pause_ns < 1024) pause_ns *= 2;
    }
    if (ok) {
        __threadfence_system();                                       // payload written before the flag is visible now
        if (arrived) arrived[s] = epoch;
    } else if (status) {
        atomicOr(status, EP_STATUS_TIMEOUT);
    }
}

__global__ void post_flags_kernel(uint32_t *flags, int first, int n, uint32_t epoch)
{
    const int s = threadIdx.x;
    if (s >= n) return;
    __threadfence_system();                                           // everything before this kernel in the stream is visible first
    asm volatile("st.volatile.global.u32 [%0], %1;" ::"l"(flags + first + s), "r"(epoch) : "memory");
}

}  // namespace
}  // namespace ep

extern "C" int ep_wait_senders(const uint32_t *flags, int num_senders, uint32_t epoch, uint64_t timeout_ns,
                               uint32_t *arrived, int32_t *status, void *stream)
{
    using namespace ep;
    if (!flags) return EP_ERR_NULL;
    if (num_senders < 1 || num_senders > kMaxSenders || timeout_ns == 0 || timeout_ns > kMaxTimeoutNs)
        return EP_ERR_INVALID_ARG;
    wait_senders_kernel<<<1, kMaxSenders, 0, static_cast<cudaStream_t>(stream)>>>(flags, num_senders, epoch, timeout_ns,
                                                                                 arrived, status);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

extern "C" int ep_post_flags(uint32_t *flags, int first_sender, int num_senders, uint32_t epoch, void *stream)
{
    using namespace ep;
    if (!flags) return EP_ERR_NULL;
    if (first_sender < 0 || num_senders < 1 || first_sender + num_senders > kMaxSenders) return EP_ERR_INVALID_ARG;
    post_flags_kernel<<<1, kMaxSenders, 0, static_cast<cudaStream_t>(stream)>>>(flags, first_sender, num_senders, epoch);
    EP_LAUNCH_CHECK(1);
    return EP_OK;
}

extern "C" int ep_host_roundtrip(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                                 const int32_t *rank_row_offsets_host, void *staging, int64_t staging_capacity_rows,
                                 void *bounce_host, int round, void *recv, int chunks_per_rank, int duplex,
                                 int32_t *status, void *stream_up_, void *stream_down_)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x || !recv_slot || !rank_row_offsets_host || !staging || !bounce_host || !recv) return EP_ERR_NULL;
    if (!aligned16(x) || !aligned16(staging) || !aligned16(recv) || staging_capacity_rows < 0 || chunks_per_rank < 1 ||
        chunks_per_rank > 64 || round < 0)
        return EP_ERR_INVALID_ARG;
    const int R = shape->num_ranks;
    if (rank_row_offsets_host[0] != 0 || rank_row_offsets_host[R] > staging_capacity_rows) return EP_ERR_CAPACITY;
    for (int r = 0; r < R; ++r)
        if (rank_row_offsets_host[r + 1] < rank_row_offsets_host[r]) return EP_ERR_INVALID_ARG;
    cudaStream_t up = static_cast<cudaStream_t>(stream_up_), down = static_cast<cudaStream_t>(stream_down_);
    cudaEvent_t *ev = nullptr;
    std::unique_lock<std::mutex> hold;
    rc = order_events(&ev, R * chunks_per_rank + 2, hold);
    if (rc != EP_OK) return rc;
    const size_t row_bytes = (size_t)shape->hidden * 2;
    // two bounce buffers alternate by round, so a buffer is reused only every other round
    char *bounce = static_cast<char *>(bounce_host) + (size_t)(round & 1) * (size_t)staging_capacity_rows * row_bytes;

    // the download stream must not run ahead of what the caller queued on the upload stream
    EP_CUDA_TRY(cudaEventRecord(ev[0], down));
    EP_CUDA_TRY(cudaStreamWaitEvent(up, ev[0], 0));
    rc = launch_dispatch(*shape, x, recv_slot, staging, staging_capacity_rows, status, up);    // pack on the SMs
    if (rc != EP_OK) return rc;
    int n_ev = 1;
    for (int phase = 0; phase < (duplex ? 1 : 2); ++phase)
        for (int r = 0; r < R; ++r) {
            const int64_t lo = rank_row_offsets_host[r], hi = rank_row_offsets_host[r + 1];
            for (int c = 0; c < chunks_per_rank; ++c) {
                const int64_t a = lo + (hi - lo) * c / chunks_per_rank, b = lo + (hi - lo) * (c + 1) / chunks_per_rank;
                if (b <= a) continue;
                const size_t off = (size_t)a * row_bytes, len = (size_t)(b - a) * row_bytes;
                if (duplex || phase == 0)      // upload: device staging -> host bounce buffer
                    EP_CUDA_TRY(cudaMemcpyAsync(bounce + off, static_cast<const char *>(staging) + off, len,
                                                cudaMemcpyDeviceToHost, up));
                if (duplex) {                  // this chunk's download may start as soon as its upload is done
                    EP_CUDA_TRY(cudaEventRecord(ev[n_ev], up));
                    EP_CUDA_TRY(cudaStreamWaitEvent(down, ev[n_ev], 0));
                    ++n_ev;
                }
                if (duplex || phase == 1)      // download: host bounce buffer -> device receive buffer
                    EP_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(recv) + off, bounce + off, len,
                                                cudaMemcpyHostToDevice, down));
            }
            if (!duplex && phase == 0 && r == R - 1) {   // serial form: all uploads, then all downloads
                EP_CUDA_TRY(cudaEventRecord(ev[n_ev], up));
                EP_CUDA_TRY(cudaStreamWaitEvent(down, ev[n_ev], 0));
                ++n_ev;
            }
        }
    return EP_OK;
}
