// Per-sender completion flags with bounded polling, and the host-staged transfers that
// use separate upload / download streams: the dispatch round trip, the same round trip
// with one consumer launch per sender, and the combine return leg with the reduction
// on the SMs.
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

// Writes the global nanosecond timer to *p: progress stamps of the per-sender pipelines.
__global__ void stamp_kernel(unsigned long long *p) { *p = global_timer_ns(); }

__global__ void post_flags_kernel(uint32_t *flags, int first, int n, uint32_t epoch)
{
    const int s = threadIdx.x;
    if (s >= n) return;
    __threadfence_system();                                           // everything before this kernel in the stream is visible first
    asm volatile("st.volatile.global.u32 [%0], %1;" ::"l"(flags + first + s), "r"(epoch) : "memory");
}

// Ordering at the start of a call that writes one half of a two-half bounce buffer. With caller
// events: wait, on the upload stream, for the event recorded when that half was last read out (two
// rounds ago), so that this round's uploads overlap the previous round's downloads. Without: wait for
// everything queued on the download stream (no overlap between rounds, always safe).
int begin_round(cudaEvent_t *pool, void *const *half_free_events, int round, cudaStream_t up, cudaStream_t down)
{
    if (half_free_events) {
        EP_CUDA_TRY(cudaStreamWaitEvent(up, static_cast<cudaEvent_t>(half_free_events[round & 1]), 0));
    } else {
        EP_CUDA_TRY(cudaEventRecord(pool[0], down));
        EP_CUDA_TRY(cudaStreamWaitEvent(up, pool[0], 0));
    }
    return EP_OK;
}

int end_round(void *const *half_free_events, int round, cudaStream_t down)
{
    if (half_free_events) EP_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(half_free_events[round & 1]), down));
    return EP_OK;
}

int check_segments(const int32_t *so, int R, int64_t capacity_rows)
{
    // src_row_offsets [R][R+1]: non-decreasing along a row, rows abut, the last entry fits the buffers
    if (so[0] != 0) return EP_ERR_INVALID_ARG;
    for (int r = 0; r < R; ++r) {
        for (int s = 0; s < R; ++s)
            if (so[r * (R + 1) + s + 1] < so[r * (R + 1) + s]) return EP_ERR_INVALID_ARG;
        if (r + 1 < R && so[(r + 1) * (R + 1)] != so[r * (R + 1) + R]) return EP_ERR_INVALID_ARG;
    }
    if (so[(R - 1) * (R + 1) + R] > capacity_rows) return EP_ERR_CAPACITY;
    return EP_OK;
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
                                 int32_t *status, void *stream_up_, void *stream_down_, void *const *half_free_events)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x || !recv_slot || !rank_row_offsets_host || !staging || !bounce_host || !recv) return EP_ERR_NULL;
    if (half_free_events && (!half_free_events[0] || !half_free_events[1])) return EP_ERR_NULL;
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

    rc = begin_round(ev, half_free_events, round, up, down);
    if (rc != EP_OK) return rc;
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
    return end_round(half_free_events, round, down);
}

// One (holder rank r, peer rank s) segment of the receive space through the bounce buffer: upload on
// `up`; download on `down` behind an event (duplex) or later (serial, phase 1).
namespace ep {
namespace {
struct Trip {
    const int32_t *so;
    int R;
    size_t row_bytes;
    char *bounce;
    const char *src;
    char *dst;
    cudaStream_t up, down;
    cudaEvent_t *ev;
    int n_ev;
    bool duplex, local_on_device;

    // phase 0: uploads (and, duplex, the downloads right behind them); phase 1: downloads of the serial form
    int move(int r, int s, int phase)
    {
        return move_rows(so[r * (R + 1) + s], so[r * (R + 1) + s + 1], local_on_device && r == s, phase);
    }
    // the same for the whole partition of holder rank r (its R segments are contiguous)
    int move_partition(int r, int phase) { return move_rows(so[r * (R + 1)], so[r * (R + 1) + R], false, phase); }

    int move_rows(int64_t a, int64_t b, bool local, int phase)
    {
        if (b <= a) return EP_OK;
        const size_t off = (size_t)a * row_bytes, len = (size_t)(b - a) * row_bytes;
        if (local) {                                   // holder and peer are the same rank: never crosses the link
            if (phase == 0) EP_CUDA_TRY(cudaMemcpyAsync(dst + off, src + off, len, cudaMemcpyDeviceToDevice, up));
            return EP_OK;
        }
        if (phase == 0) EP_CUDA_TRY(cudaMemcpyAsync(bounce + off, src + off, len, cudaMemcpyDeviceToHost, up));
        if (duplex) {
            EP_CUDA_TRY(cudaEventRecord(ev[n_ev], up));
            EP_CUDA_TRY(cudaStreamWaitEvent(down, ev[n_ev], 0));
            ++n_ev;
        }
        if (duplex || phase == 1) EP_CUDA_TRY(cudaMemcpyAsync(dst + off, bounce + off, len, cudaMemcpyHostToDevice, down));
        return EP_OK;
    }
    // `down` continues only after everything queued on `up` so far (device-side copies of local segments included)
    int join()
    {
        EP_CUDA_TRY(cudaEventRecord(ev[n_ev], up));
        EP_CUDA_TRY(cudaStreamWaitEvent(down, ev[n_ev], 0));
        ++n_ev;
        return EP_OK;
    }
};
}  // namespace
}  // namespace ep

extern "C" int ep_host_dispatch_per_sender(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                                           const int32_t *pair_slot, const int32_t *src_row_offsets_host,
                                           void *staging, void *recv, int64_t capacity_rows, void *bounce_host,
                                           int round, void *grouped, int64_t grouped_capacity_rows,
                                           const uint32_t *sender_flags, uint32_t epoch, uint64_t timeout_ns,
                                           uint32_t *arrived, uint64_t *stamps_ns, int flags, int32_t *status,
                                           void *stream_up_, void *stream_down_, void *stream_consume_,
                                           void *const *half_free_events)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!x || !recv_slot || !pair_slot || !src_row_offsets_host || !staging || !recv || !bounce_host || !grouped)
        return EP_ERR_NULL;
    if (half_free_events && (!half_free_events[0] || !half_free_events[1])) return EP_ERR_NULL;
    if (!aligned16(x) || !aligned16(staging) || !aligned16(recv) || !aligned16(grouped) || capacity_rows < 0 ||
        grouped_capacity_rows < 0 || round < 0 || (flags & ~(EP_HOST_DUPLEX | EP_HOST_PER_PEER | EP_HOST_LOCAL_ON_DEVICE)))
        return EP_ERR_INVALID_ARG;
    if (sender_flags && (timeout_ns == 0 || timeout_ns > kMaxTimeoutNs)) return EP_ERR_INVALID_ARG;
    const int R = shape->num_ranks, K = shape->top_k, Tr = shape->num_tokens / R;
    rc = check_segments(src_row_offsets_host, R, capacity_rows);
    if (rc != EP_OK) return rc;
    cudaStream_t up = static_cast<cudaStream_t>(stream_up_), down = static_cast<cudaStream_t>(stream_down_),
                 cons = static_cast<cudaStream_t>(stream_consume_);
    cudaEvent_t *ev = nullptr;
    std::unique_lock<std::mutex> hold;
    rc = order_events(&ev, R * R + 3 * R + 4, hold);
    if (rc != EP_OK) return rc;
    const size_t row_bytes = (size_t)shape->hidden * 2;
    const bool duplex = flags & EP_HOST_DUPLEX, per_sender = flags & EP_HOST_PER_PEER;
    Trip trip{src_row_offsets_host, R, row_bytes,
              static_cast<char *>(bounce_host) + (size_t)(round & 1) * (size_t)capacity_rows * row_bytes,
              static_cast<const char *>(staging), static_cast<char *>(recv), up, down, ev, 1, duplex,
              (flags & EP_HOST_LOCAL_ON_DEVICE) != 0};

    rc = begin_round(ev, half_free_events, round, up, down);
    if (rc != EP_OK) return rc;
    // the consumer stream starts behind what is queued on the upload stream now (the caller's x) and must have
    // finished with `grouped`/`recv` of the previous call before this call's downloads overwrite `recv`
    EP_CUDA_TRY(cudaEventRecord(ev[trip.n_ev], cons));
    EP_CUDA_TRY(cudaStreamWaitEvent(down, ev[trip.n_ev], 0));
    ++trip.n_ev;
    if (stamps_ns) {
        stamp_kernel<<<1, 1, 0, up>>>(reinterpret_cast<unsigned long long *>(stamps_ns));
        EP_LAUNCH_CHECK(1);
    }
    rc = launch_dispatch(*shape, x, recv_slot, staging, capacity_rows, status, up);        // pack on the SMs
    if (rc != EP_OK) return rc;

    // the consumer of sender s: local grouping of the pairs of s's tokens, recv rows -> pair rows
    auto consume = [&](int s) -> int {
        if (sender_flags) {                      // gate on the sender's completion flag, bounded
            wait_senders_kernel<<<1, kMaxSenders, 0, cons>>>(sender_flags + s, 1, epoch, timeout_ns,
                                                             arrived ? arrived + s : nullptr, status);
            EP_LAUNCH_CHECK(1);
        }
        int rc2 = launch_permute(shape->hidden, recv, capacity_rows, recv_slot + (size_t)s * Tr * K, grouped,
                                 grouped_capacity_rows, pair_slot + (size_t)s * Tr * K, (int64_t)Tr * K, status, cons);
        if (rc2 != EP_OK) return rc2;
        if (stamps_ns) {
            stamp_kernel<<<1, 1, 0, cons>>>(reinterpret_cast<unsigned long long *>(stamps_ns) + 1 + s);
            EP_LAUNCH_CHECK(1);
        }
        return EP_OK;
    };
    // after sender s's last segment has been queued for download: release (or not yet) its consumer
    auto sender_done = [&](int s) -> int {
        if (trip.local_on_device && duplex) {      // the device-side copy of the local segment ran on `up`
            int rc2 = trip.join();
            if (rc2 != EP_OK) return rc2;
        }
        if (!per_sender && s != R - 1) return EP_OK;
        EP_CUDA_TRY(cudaEventRecord(ev[trip.n_ev], down));
        EP_CUDA_TRY(cudaStreamWaitEvent(cons, ev[trip.n_ev], 0));
        ++trip.n_ev;
        if (per_sender) return consume(s);
        for (int q = 0; q < R; ++q) {            // wait-for-all policy: every consumer behind the last download
            int rc2 = consume(q);
            if (rc2 != EP_OK) return rc2;
        }
        return EP_OK;
    };

    for (int s = 0; s < R; ++s) {                // sender-major: a sender's segments for every destination, then the next sender
        for (int r = 0; r < R; ++r)
            if ((rc = trip.move(r, s, 0)) != EP_OK) return rc;
        if (duplex && (rc = sender_done(s)) != EP_OK) return rc;
    }
    if (!duplex) {
        if ((rc = trip.join()) != EP_OK) return rc;
        for (int s = 0; s < R; ++s) {
            for (int r = 0; r < R; ++r)
                if ((rc = trip.move(r, s, 1)) != EP_OK) return rc;
            if ((rc = sender_done(s)) != EP_OK) return rc;
        }
    }
    return end_round(half_free_events, round, down);
}

extern "C" int ep_host_combine(const ep_shape_t *shape, const void *out, int64_t out_rows, const int32_t *pair_slot,
                               const int32_t *recv_slot, const float *topk_weights,
                               const int32_t *src_row_offsets_host, void *partial_send, void *partial_recv,
                               int64_t partial_capacity_rows, void *bounce_host, int round, void *y, int flags,
                               int32_t *status, void *stream_up_, void *stream_down_,
                               void *const *half_free_events)
{
    using namespace ep;
    int rc = check_shape(shape, true);
    if (rc != EP_OK) return rc;
    if (shape->num_tokens == 0) return EP_OK;
    if (!out || !pair_slot || !recv_slot || !topk_weights || !src_row_offsets_host || !partial_send || !partial_recv ||
        !bounce_host || !y)
        return EP_ERR_NULL;
    if (half_free_events && (!half_free_events[0] || !half_free_events[1])) return EP_ERR_NULL;
    if (!aligned16(out) || !aligned16(partial_send) || !aligned16(partial_recv) || !aligned16(y) || out_rows < 0 ||
        partial_capacity_rows < 0 || round < 0 || (flags & ~(EP_HOST_DUPLEX | EP_HOST_PER_PEER | EP_HOST_LOCAL_ON_DEVICE)))
        return EP_ERR_INVALID_ARG;
    const int R = shape->num_ranks, K = shape->top_k, H = shape->hidden, Tr = shape->num_tokens / R;
    rc = check_segments(src_row_offsets_host, R, partial_capacity_rows);
    if (rc != EP_OK) return rc;
    cudaStream_t up = static_cast<cudaStream_t>(stream_up_), down = static_cast<cudaStream_t>(stream_down_);
    cudaEvent_t *ev = nullptr;
    std::unique_lock<std::mutex> hold;
    rc = order_events(&ev, R * R + 2 * R + 4, hold);
    if (rc != EP_OK) return rc;
    const size_t row_bytes = (size_t)H * 2;
    const bool duplex = flags & EP_HOST_DUPLEX, per_owner = flags & EP_HOST_PER_PEER;
    Trip trip{src_row_offsets_host, R, row_bytes,
              static_cast<char *>(bounce_host) + (size_t)(round & 1) * (size_t)partial_capacity_rows * row_bytes,
              static_cast<const char *>(partial_send), static_cast<char *>(partial_recv), up, down, ev, 1, duplex,
              (flags & EP_HOST_LOCAL_ON_DEVICE) != 0};

    rc = begin_round(ev, half_free_events, round, up, down);
    if (rc != EP_OK) return rc;
    // every expert rank sums what it computed for a token into one row: these rows are what travels
    rc = launch_partial_rows(*shape, out, out_rows, pair_slot, recv_slot, 0, topk_weights, partial_send,
                             partial_capacity_rows, status, up);
    if (rc != EP_OK) return rc;

    // the owner's reduction on the SMs: tokens of owner s (or all tokens) once their blocks are down
    auto reduce = [&](int s_lo, int s_hi) -> int {
        return launch_sum_partial_rows(H, K, partial_recv, partial_capacity_rows, recv_slot + (size_t)s_lo * Tr * K,
                                       static_cast<uint16_t *>(y) + (size_t)s_lo * Tr * H, (s_hi - s_lo) * Tr, status, down);
    };
    auto owner_done = [&](int s) -> int {
        if (trip.local_on_device && duplex) {
            int rc2 = trip.join();
            if (rc2 != EP_OK) return rc2;
        }
        if (per_owner) return reduce(s, s + 1);
        return s == R - 1 ? reduce(0, R) : EP_OK;
    };
    if (!per_owner && !trip.local_on_device) {
        // one reduction at the end and every block over the link: an expert rank's R blocks are contiguous, so
        // they travel as one piece (R pieces instead of R*R: the fewest that keep both directions busy)
        for (int phase = 0; phase < (duplex ? 1 : 2); ++phase) {
            if (phase == 1 && (rc = trip.join()) != EP_OK) return rc;
            for (int r = 0; r < R; ++r)
                if ((rc = trip.move_partition(r, phase)) != EP_OK) return rc;
        }
        if ((rc = reduce(0, R)) != EP_OK) return rc;
        return end_round(half_free_events, round, down);
    }
    for (int s = 0; s < R; ++s) {                // owner-major: every expert rank's block for owner s, then the next owner
        for (int r = 0; r < R; ++r)
            if ((rc = trip.move(r, s, 0)) != EP_OK) return rc;
        if (duplex && (rc = owner_done(s)) != EP_OK) return rc;
    }
    if (!duplex) {
        if ((rc = trip.join()) != EP_OK) return rc;
        for (int s = 0; s < R; ++s) {
            for (int r = 0; r < R; ++r)
                if ((rc = trip.move(r, s, 1)) != EP_OK) return rc;
            if ((rc = owner_done(s)) != EP_OK) return rc;
        }
    }
    return end_round(half_free_events, round, down);
}
