/*
 * ep.h -- C ABI of the B200 (sm_100a) routing-aware expert-parallel token
 * dispatch / combine library.
 *
 * The problem, as the paper states it (Section 2.1, "Distributed MoE and expert
 * parallelism"): a router picks K of E experts for each of T tokens; the experts
 * are partitioned over R devices ("ranks") and every rank owns a block of the
 * tokens. Before the expert computation a token's activation must reach every
 * rank that hosts one of its picked experts (dispatch); afterwards the expert
 * outputs return to the token's owner and are summed there (combine). This
 * library implements the routing-aware form (Section 2.1, "Communication
 * patterns of dispatch and combine"; Section 4.5, "Routing-aware
 * communication"): only the rows a destination needs are moved, once per
 * destination rank. The R ranks are logical partitions of one GPU's buffers (or
 * of a mapped pinned host buffer standing in for the CPU bounce buffer of
 * Section 4.2).
 *
 * Conventions
 *   - rank of expert e:  e / (E/R)     source rank of token t:  t / (T/R)
 *   - pair order: (t,k) < (t',k')  iff  t < t' or (t == t' and k < k')
 *   - an entry topk_idx[t][k] == -1 is masked and skipped everywhere
 *   - receive space: one row per distinct (token, destination rank); rank r owns
 *     rows [rank_row_offsets[r], rank_row_offsets[r+1]), ordered by token
 *   - pair space: one entry per valid (t,k), grouped by expert id, ordered by
 *     (t,k) inside an expert; rank r owns entries
 *     [expert_offsets[r*E/R], expert_offsets[(r+1)*E/R])
 *
 * Every function returns EP_OK (0) or a negative ep_error_t. No function
 * allocates device memory, prints, throws or aborts. State the library keeps
 * between calls: the last CUDA error code, a launch counter, per-device one-time
 * kernel attributes, and the event pool of the multi-stream host-staged calls. Unless stated otherwise a
 * function only enqueues work on `stream` (a cudaStream_t passed as void*; NULL
 * is the default stream) and does not synchronise. "device" pointers must be
 * valid on the current CUDA device; the caller owns every buffer.
 *
 * Shape limits, checked on the host before anything is launched
 * (EP_ERR_INVALID_ARG otherwise): T >= 0, T % R == 0, T*K < 2^31; 1 <= K <= 32;
 * 1 <= R <= 64; E % R == 0, R <= E <= 4096; H >= 8 and H % 8 == 0 (rows are
 * whole 16-byte vectors); bf16 buffers 16-byte aligned.
 */
#ifndef EP_B200_H
#define EP_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EP_OK = 0,
    EP_ERR_NULL = -1,         /* a required pointer is NULL */
    EP_ERR_INVALID_ARG = -2,  /* shape outside the limits above, misaligned buffer */
    EP_ERR_CAPACITY = -3,     /* workspace / arena / staging buffer too small */
    EP_ERR_CUDA = -4,         /* a CUDA runtime call failed: see ep_last_cuda_error */
    EP_ERR_STATIC_SCRATCH = -5 /* ep_layout_static: the shape needs more scratch than the fixed array holds */
} ep_error_t;

/* bits of the device status word */
#define EP_STATUS_BAD_INDEX 1 /* an expert id outside [-1, E) was seen and masked */
#define EP_STATUS_CAPACITY  2 /* a slot >= the buffer's row capacity was skipped  */
#define EP_STATUS_TIMEOUT   4 /* ep_wait_senders gave up on at least one sender     */

typedef struct {
    int32_t num_tokens;  /* T */
    int32_t top_k;       /* K */
    int32_t hidden;      /* H, bf16 elements per row */
    int32_t num_experts; /* E */
    int32_t num_ranks;   /* R */
} ep_shape_t;

/* Outputs of ep_layout: device pointers to caller-allocated int32 arrays. */
typedef struct {
    int32_t *expert_counts;    /* [E]         valid pairs per expert                           */
    int32_t *expert_offsets;   /* [E+1]       exclusive scan of expert_counts; [E] = P         */
    int32_t *rank_rows;        /* [R]         distinct tokens that reach rank r                */
    int32_t *rank_row_offsets; /* [R+1]       exclusive scan of rank_rows; [R] = N_recv        */
    int32_t *src_row_offsets;  /* [R*(R+1)]   [r][s] = first receive row of source rank s
                                              inside rank r; [r][R] = end of rank r           */
    int32_t *recv_slot;        /* [T*K]       receive row of pair (t,k); -1 if masked          */
    int32_t *pair_slot;        /* [T*K]       pair-space index of (t,k); -1 if masked          */
    int32_t *recv_token;       /* [T*min(K,R)] receive row -> token (first N_recv entries)     */
    int32_t *pair_row;         /* [T*K]       pair-space index -> receive row (first P)        */
    int32_t *pair_token;       /* [T*K]       pair-space index -> token (first P)              */
    int32_t *status;           /* [1]         EP_STATUS_* bits, rewritten by every ep_layout   */
} ep_layout_t;

/*
 * Layout (Section 2.1: which devices a token must reach; Section 4.3: each
 * device groups what it received by the experts it owns; Section 4.4: a
 * receiver may start on each sender's portion separately, hence
 * src_row_offsets). Computes every array of ep_layout_t from topk_idx
 * [T][K] (device, int32, row-major) entirely on the device: the routing table
 * never travels to the host (Section 4.5 names that round trip as what made
 * routing-aware transfers slow).
 *
 * `workspace` (device, 16-byte aligned) must hold ep_layout_workspace_bytes()
 * bytes; its contents need no initialisation and are garbage afterwards. Calls
 * that share a workspace must be stream-ordered. T == 0 writes the (all-zero)
 * counts and offsets and touches nothing else.
 * Errors: EP_ERR_NULL, EP_ERR_INVALID_ARG, EP_ERR_CAPACITY (workspace), EP_ERR_CUDA.
 */
size_t ep_layout_workspace_bytes(const ep_shape_t *shape);
int ep_layout(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
              void *workspace, size_t workspace_bytes, void *stream);

/*
 * The two halves of ep_layout as separate calls, so that they can run on
 * different streams: dispatch needs only the receive-row half, combine only the
 * pair half, and the pair half can therefore be computed while dispatch moves
 * rows (Section 4.5 blames the routing-metadata step for the cost of
 * routing-aware transfers; this takes most of it off the critical path).
 *   ep_layout_ranks  writes rank_rows, rank_row_offsets, src_row_offsets,
 *                    recv_slot, recv_token and status;
 *   ep_layout_pairs  writes expert_counts, expert_offsets, pair_slot, pair_row
 *                    and pair_token, and never touches status.
 * Each reads only topk_idx; the fields of `out` a call does not write may be
 * NULL. Together they produce exactly what ep_layout produces. Calls that may
 * overlap need workspaces of their own (ep_layout_workspace_bytes each).
 */
int ep_layout_ranks(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                    void *workspace, size_t workspace_bytes, void *stream);
int ep_layout_pairs(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * Layout without any allocation (the paper has no counterpart; this entry point
 * exists for integration reasons only). Some callers cannot obtain device
 * memory at the point where they need a layout: code running inside a serving
 * engine whose memory pool is fully handed out, a plugin that is forbidden to
 * call cudaMalloc, a component that must not disturb a caching allocator. For
 * them this call computes exactly what ep_layout computes -- same arguments
 * minus the workspace, same outputs bit for bit, same errors -- but takes its
 * scratch from a fixed array of EP_LAYOUT_STATIC_SCRATCH_BYTES bytes that lives
 * inside the library on every GPU that loads it, until the process exits. It
 * calls no cudaMalloc, cudaFree or other allocating routine. The caller still
 * provides topk_idx and every output array.
 *
 *   - Limit: the scratch a shape needs is ep_layout_workspace_bytes(shape): 16
 *     bytes up to 256 tokens, else 4*(E+R+1) bytes per CTA of 256 tokens (fewer
 *     tokens when large E or K shrink the CTA, more once there would be over
 *     128 CTAs; 34 KB for T=8192, E=256, R=8). Shapes that need more than the
 *     array holds return EP_ERR_STATIC_SCRATCH and enqueue nothing.
 *   - First call on a device: looks up the array's device address (once per
 *     device, with that device current). Make that first call outside any
 *     stream capture.
 *   - The array is shared by every call on that device and keeps what the last
 *     call left in it; the kernels rewrite all they read, so no clearing is
 *     needed. Two calls that overlap on the GPU (different streams, no ordering)
 *     race on it: order them.
 */
#define EP_LAYOUT_STATIC_SCRATCH_BYTES (1u << 20)
size_t ep_layout_static_scratch_bytes(void);
int ep_layout_static(const ep_shape_t *shape, const int32_t *topk_idx, const ep_layout_t *out,
                     void *stream);

/*
 * Dispatch (Section 1 and Section 2.1: activations go to the devices holding the
 * selected experts, one copy per destination device): for every valid pair
 * recv[recv_slot[t][k]][0..H) = x[t][0..H), bit for bit. x is [T][H] bf16
 * (device). recv is [recv_capacity_rows][H] bf16, device memory or the device
 * alias of mapped pinned host memory. A row is written once per (token, rank).
 * Rows no pair names are not touched. A slot >= recv_capacity_rows is skipped
 * and sets EP_STATUS_CAPACITY in *status (device, may be NULL; bits are OR-ed
 * in, never cleared here).
 */
int ep_dispatch(const ep_shape_t *shape, const void *x, const int32_t *recv_slot, void *recv,
                int64_t recv_capacity_rows, int32_t *status, void *stream);

/*
 * Layout and dispatch in one call (Section 4.5: at decode sizes the transfers are
 * a few kilobytes and the cost is latency and synchronisation, not bytes; the
 * routing-metadata step is what made routing-aware transfers slow). Produces
 * exactly what ep_layout followed by ep_dispatch (with status = out->status)
 * produces: every array of `out`, the dispatched rows in recv, and the status
 * word (EP_STATUS_BAD_INDEX, EP_STATUS_CAPACITY when N_recv exceeds
 * recv_capacity_rows). The call runs the layout kernels and then the dispatch
 * kernel, launched so that its CTAs load their rows of x while the layout still
 * runs (x and topk_idx are inputs of this call: they must be complete on
 * `stream` before it). Only batches of up to 1024 tokens that the layout's
 * fastest kernels do not cover (a top-k of 9 or above 10, more than 1024
 * experts, tables that are not 16-byte aligned) and whose routing table fits in
 * shared memory take one launch in which every CTA derives the layout for itself
 * and moves its own tokens' rows. stream_pairs (may be NULL) is a second
 * stream for batches of more than 1024 tokens: the pair half of the layout,
 * which dispatch does not need, then runs there beside dispatch; the call
 * orders it behind what is queued on `stream` and makes `stream` wait for it at
 * the end, so that on return everything is ordered on `stream` as if it had run
 * there. With stream_pairs such a batch needs a workspace of
 * 2 * ep_layout_workspace_bytes() + 256 bytes (EP_ERR_CAPACITY otherwise);
 * batches of up to 1024 tokens ignore stream_pairs and need the plain size.
 * The two ordering events come from the library's pool (see the host-staged
 * conventions below).
 */
int ep_layout_dispatch(const ep_shape_t *shape, const int32_t *topk_idx, const void *x, const ep_layout_t *out,
                       void *workspace, size_t workspace_bytes, void *recv, int64_t recv_capacity_rows,
                       void *stream, void *stream_pairs);

/*
 * Combine (Section 1; Section 4.3: the contributions that arrive for a token are
 * added on an SM): y[t][h] = bf16( sum_k w[t][k] * out[slot[t][k]][h] ), an fp32
 * fused multiply-add chain from +0 in ascending k, pairs with slot -1 skipped,
 * one round-to-nearest-even narrowing at the end. out is [out_rows][H] bf16
 * (device); slot [T][K] int32 is either pair_slot (out holds one row per pair)
 * or recv_slot (out is a receive buffer); topk_weights [T][K] fp32; y [T][H]
 * bf16. A slot >= out_rows is skipped and sets EP_STATUS_CAPACITY in *status
 * (device, may be NULL).
 */
int ep_combine(const ep_shape_t *shape, const void *out, int64_t out_rows, const int32_t *slot,
               const float *topk_weights, void *y, int32_t *status, void *stream);

/*
 * Local grouping by expert (Section 4.3: the receiver reorders what it received
 * by the experts it owns, a permutation that stays on the SMs):
 * grouped[p] = recv[pair_row[p]]
 * for p < P, where P is read on the device from expert_offsets[E]. grouped is
 * [grouped_capacity_rows][H] bf16 (device); entries p >= capacity are skipped
 * with EP_STATUS_CAPACITY.
 */
int ep_group(const ep_shape_t *shape, const void *recv, int64_t recv_rows, const int32_t *pair_row,
             const int32_t *expert_offsets, void *grouped, int64_t grouped_capacity_rows,
             int32_t *status, void *stream);

/*
 * Combine with partial outputs (Section 2.1, "Communication patterns of dispatch
 * and combine": in the All-to-Allv form what returns to the owner is one partial
 * output per rank the token reached): every rank
 * first sums, per token it received, the weighted outputs of its own experts
 * into one row of `partial` (receive space, [partial_capacity_rows][H] bf16):
 *   partial[recv_slot[t][k]] = bf16( fp32 fma chain over the k' (ascending) that
 *                                    share this receive row of w[t][k']*out[pair_slot[t][k']] )
 * and the owner adds a token's distinct partial rows in the order of their first k:
 *   y[t] = bf16( fp32 sum from +0 ).
 * Two roundings to bf16 instead of one: the result differs from ep_combine by at
 * most one bf16 half-ulp per partial row. Rows of `partial` no token names are
 * not touched. Out-of-range slots are skipped with EP_STATUS_CAPACITY.
 */
int ep_combine_partial(const ep_shape_t *shape, const void *out, int64_t out_rows,
                       const int32_t *pair_slot, const int32_t *recv_slot, const float *topk_weights,
                       void *partial, int64_t partial_capacity_rows, void *y, int32_t *status,
                       void *stream);

/*
 * Dense formulation on the same logical ranks (Section 2.1: All-Gather and
 * Reduce-Scatter, Figure 3; Section 4.2: the volumes 2(N-1)S and N*S), the
 * baseline the routing-aware path is compared with.
 * ep_dense_allgather: gathered[r*T + t] = x[t] for every rank r: R*T rows
 * whatever the routing (gathered is [R*T][H] bf16, device).
 * ep_dense_reduce_scatter: rank r's dense buffer ordered by source token,
 *   dense[r*T + t] = bf16( fma chain over the k (ascending) whose expert lives on r ),
 * +0 where the token has no expert on r, then y[t] = bf16( fp32 sum over
 * r = 0..R-1 of dense[r*T + t] ). dense is [R*T][H] bf16 (device), fully
 * written. Needs R <= 32.
 */
int ep_dense_allgather(const ep_shape_t *shape, const void *x, void *gathered, void *stream);
int ep_dense_reduce_scatter(const ep_shape_t *shape, const int32_t *topk_idx, const void *out,
                            int64_t out_rows, const int32_t *pair_slot, const float *topk_weights,
                            void *dense, void *y, int32_t *status, void *stream);

/*
 * Host-staged dispatch, copy-engine arm (Section 2.2 and Section 4.3: the DMA
 * engines move contiguous regions only, so routing-dependent rows are first
 * packed by a kernel): ep_dispatch into `staging` (device,
 * [staging_capacity_rows][H]) followed by cudaMemcpyAsync device-to-host copies
 * into recv_host (pinned host memory, same row layout) on the same stream. With
 * rank_row_offsets_host (host, [R+1]) one copy per destination rank's partition
 * is issued; with NULL a single copy of staging_capacity_rows rows (no row count
 * ever reaches the host).
 */
int ep_dispatch_copy_engine(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                            const int32_t *rank_row_offsets_host, void *staging,
                            int64_t staging_capacity_rows, void *recv_host, int32_t *status,
                            void *stream);

/*
 * Host-staged transfers on two streams: shared conventions of ep_host_roundtrip,
 * ep_host_dispatch_per_sender and ep_host_combine.
 *
 *   - Bounce buffer (Section 4.2: the pinned host buffer every device writes once
 *     and the others read; Section 4.4: two buffers alternate): bounce_host is
 *     pinned host memory of 2 * capacity_rows rows of H bf16; a call uses the half
 *     `round & 1`, at the same row offsets as the device buffers.
 *   - Streams (Section 4.3: uploads and downloads are issued on two different
 *     streams and cut into pieces, so that both directions of the host link are
 *     busy): device-to-host copies and the packing / partial-sum kernel run on
 *     stream_up, host-to-device copies and what consumes them on stream_down (and
 *     stream_consume). Inputs must be complete on stream_up; results are complete
 *     when stream_down (and stream_consume) are.
 *   - Reuse of a half (Section 4.4: a buffer is reused only after its readers are
 *     done with it): half_free_events is NULL or an array of two cudaEvent_t the
 *     caller created (passed as void*). Given, a call waits on stream_up for
 *     half_free_events[round & 1] before it writes the half and records that event
 *     on stream_down after its last read of it; so round n+1's uploads overlap
 *     round n's downloads and round n+2 waits for round n. An event that was never
 *     recorded counts as complete. NULL: the call's uploads wait for everything
 *     queued on stream_down (no overlap between rounds, always safe).
 *   - flags: EP_HOST_DUPLEX            a piece's download is released by an event right after
 *                                      its upload (else: all uploads, then all downloads);
 *            EP_HOST_PER_PEER          the consumer is launched per peer rank as soon as that
 *                                      peer's pieces are down (Section 4.4, per-sender policy),
 *                                      else once behind the last download (global policy);
 *            EP_HOST_LOCAL_ON_DEVICE   a segment whose two ranks coincide is copied on the
 *                                      device and never crosses the host link (Section 4.2:
 *                                      only the N-1 remote shards / blocks travel).
 *   - Process-wide state: the ordering events between the streams come from a pool
 *     the library creates on first use, per device, and keeps until the process
 *     exits (events hold no device memory). A call holds the pool's lock while it
 *     enqueues, so calls from several host threads are serialised, not interleaved.
 *     The same holds for ep_host_step_pipelined.
 */
#define EP_HOST_DUPLEX          1
#define EP_HOST_PER_PEER        2
#define EP_HOST_LOCAL_ON_DEVICE 4

/*
 * Host-staged dispatch round trip. Packs the receive rows into `staging` (device)
 * with the dispatch kernel on stream_up, copies them piece by piece to the bounce
 * half and from there into `recv` (device, same row layout) on stream_down. Each
 * rank's partition [rank_row_offsets_host[r], [r+1]) (host, [R+1]) is cut into
 * chunks_per_rank pieces (1..64). duplex != 0: EP_HOST_DUPLEX as above.
 * Errors: EP_ERR_CAPACITY when the offsets exceed staging_capacity_rows.
 */
int ep_host_roundtrip(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                      const int32_t *rank_row_offsets_host, void *staging, int64_t staging_capacity_rows,
                      void *bounce_host, int round, void *recv, int chunks_per_rank, int duplex,
                      int32_t *status, void *stream_up, void *stream_down, void *const *half_free_events);

/*
 * Host-staged dispatch with per-sender completion (Section 4.4: a receiver starts
 * on each sender's data as soon as that sender is done; Section 4.5: computation
 * on a sender's activations begins while the other senders' transfers continue).
 * The pieces are the (destination r, sender s) segments
 * [src_row_offsets_host[r][s], [r][s+1]) of the receive space (host copy of the
 * layout's src_row_offsets, [R][R+1]), moved sender by sender. The consumer of
 * sender s is the local grouping of the pairs of s's tokens,
 *   grouped[pair_slot[t][k]] = recv[recv_slot[t][k]]  for t in s's block,
 * on stream_consume. EP_HOST_PER_PEER: it is launched behind sender s's last
 * download; otherwise all R consumers are launched behind the last download of
 * all. After the call recv holds the dispatched rows and grouped equals what
 * ep_group produces.
 *   sender_flags  NULL, or R completion flags (device or mapped pinned memory):
 *                 the consumer of sender s is additionally gated by a bounded wait
 *                 (as ep_wait_senders: epoch, timeout_ns <= 2 s, EP_STATUS_TIMEOUT
 *                 and fall through when it runs out) on sender_flags[s]; arrived
 *                 (device, [R], may be NULL) receives the epoch per sender. The
 *                 flags are written by the host or by earlier work; the library
 *                 never makes a kernel wait on a kernel it launches later.
 *   stamps_ns     NULL, or R+1 device words: [0] = global timer (ns) when the
 *                 pipeline starts on stream_up, [1+s] = when sender s's consumer
 *                 has finished.
 */
int ep_host_dispatch_per_sender(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                                const int32_t *pair_slot, const int32_t *src_row_offsets_host, void *staging,
                                void *recv, int64_t capacity_rows, void *bounce_host, int round, void *grouped,
                                int64_t grouped_capacity_rows, const uint32_t *sender_flags, uint32_t epoch,
                                uint64_t timeout_ns, uint32_t *arrived, uint64_t *stamps_ns, int flags,
                                int32_t *status, void *stream_up, void *stream_down, void *stream_consume,
                                void *const *half_free_events);

/*
 * Host-staged combine, the return leg (Section 4.2, reduce-scatter with GPU
 * reduction: every device uploads the blocks meant for the others, every owner
 * downloads the blocks meant for it and adds them on its SMs; Section 4.3: the
 * reduction stays on an SM; Section 4.4, Figure 10: an owner starts as soon as its
 * senders are done). Computes exactly what ep_combine_partial computes:
 *   1. on stream_up, every expert rank sums its weighted outputs per token it
 *      received into one row of partial_send (receive space, device);
 *   2. the (expert rank r, owner s) blocks [src_row_offsets_host[r][s], [r][s+1])
 *      travel owner by owner: device -> bounce half on stream_up, bounce half ->
 *      partial_recv (device) on stream_down;
 *   3. on stream_down the owner adds a token's partial rows into y:
 *      EP_HOST_PER_PEER: per owner s as soon as its R blocks are down; otherwise
 *      once for all tokens behind the last download (then, unless local blocks
 *      stay on the device, an expert rank's R blocks travel as one piece).
 * partial_send, partial_recv: [partial_capacity_rows][H] bf16 device buffers;
 * afterwards partial_recv equals the `partial` of ep_combine_partial and y its y.
 */
int ep_host_combine(const ep_shape_t *shape, const void *out, int64_t out_rows, const int32_t *pair_slot,
                    const int32_t *recv_slot, const float *topk_weights, const int32_t *src_row_offsets_host,
                    void *partial_send, void *partial_recv, int64_t partial_capacity_rows, void *bounce_host,
                    int round, void *y, int flags, int32_t *status, void *stream_up, void *stream_down,
                    void *const *half_free_events);

/*
 * Per-sender completion flags (Section 4.4: the payload stays contiguous and the
 * flags are stored apart; one thread per sender polls its flag with uncached
 * loads and pauses between attempts; a flag has a single writer, so no atomics).
 * ep_wait_senders enqueues a one-CTA kernel whose thread s polls flags[s]
 * (device memory or mapped pinned host memory) until it reads `epoch`, then
 * writes `epoch` to arrived[s] (device, may be NULL), the word consumers watch.
 * Every wait is bounded: after timeout_ns (at most 2 s) the thread gives up,
 * EP_STATUS_TIMEOUT is OR-ed into *status (device, may be NULL) and the kernel
 * ends; nothing hangs and later work on the stream still runs. 1 <= num_senders
 * <= 64. ep_post_flags enqueues the writer side: flags[first..first+n) = epoch,
 * ordered after all earlier work of its stream.
 */
int ep_wait_senders(const uint32_t *flags, int num_senders, uint32_t epoch, uint64_t timeout_ns,
                    uint32_t *arrived, int32_t *status, void *stream);
int ep_post_flags(uint32_t *flags, int first_sender, int num_senders, uint32_t epoch, void *stream);

/*
 * One whole step from host buffers: copies x, topk_idx and topk_weights from
 * (pinned) host memory to the device arena, runs layout, dispatch, local
 * grouping (the identity expert: out[p] = recv[pair_row[p]]) and combine over
 * the pair space, and copies y back. All enqueued on `stream`; the caller
 * synchronises. `arena` is device memory of ep_host_step_arena_bytes() bytes,
 * 256-byte aligned. status_host (pinned host, may be NULL) receives the device
 * status word after the step.
 */
size_t ep_host_step_arena_bytes(const ep_shape_t *shape);
int ep_host_step(const ep_shape_t *shape, const void *x_host, const int32_t *topk_idx_host,
                 const float *topk_weights_host, void *y_host, int32_t *status_host, void *arena,
                 size_t arena_bytes, void *stream);

/*
 * The same step with the host link used in both directions at once (Section 4.3:
 * uploads and downloads on separate streams, cut into chunks): the tokens are
 * cut into `chunks` contiguous chunks; chunk c's rows are uploaded on stream_in
 * while chunk c-1 runs dispatch, local grouping and combine on stream_compute
 * and chunk c-2's result is downloaded on stream_out (layout runs once, on the
 * whole routing table, before the first chunk). Results are identical to
 * ep_host_step. Complete when stream_out is. The three streams must differ for
 * any overlap; the arena may be reused by the next call without synchronising
 * (the call orders itself after the previous one). 1 <= chunks <= 256. Ordering
 * events come from the library's process-wide pool (see the host-staged
 * conventions above); calls from several host threads are serialised.
 * Steps back to back (Section 4.4: two buffers used in turn, so that a round's
 * transfers need not wait for the round before it): the arena holds two copies
 * of what the copy streams touch (x, topk_idx, topk_weights, y, the status
 * word). With step_events == NULL every call uses the first copy and waits for
 * the previous call's kernels before it uploads and for its downloads before it
 * computes. With step_events = four caller-owned cudaEvent_t (created by the
 * caller, never recorded or recorded long ago; the same four for every call on
 * this arena) call number `round` (0, 1, 2, ... consecutive) uses copy
 * round & 1 and waits only for call round - 2, which used the same copy:
 * its uploads start while the previous call's downloads are still running. The
 * call records step_events[round & 1] behind its kernels and
 * step_events[2 + (round & 1)] behind its downloads. Errors: EP_ERR_NULL for a
 * NULL entry of step_events, EP_ERR_INVALID_ARG for round < 0.
 */
int ep_host_step_pipelined(const ep_shape_t *shape, const void *x_host, const int32_t *topk_idx_host,
                           const float *topk_weights_host, void *y_host, int32_t *status_host, void *arena,
                           size_t arena_bytes, int chunks, void *stream_in, void *stream_compute,
                           void *stream_out, int round, void *const *step_events);

/* Reads a device status word: copies it to *status_host and SYNCHRONISES the stream. */
int ep_status(const int32_t *status_dev, void *stream, int32_t *status_host);

/*
 * Bandwidth probes over caller-provided buffers (no paper counterpart; they give
 * the attainable denominators beside the nominal ones). Runs `iters` repetitions
 * on `stream`, times each with CUDA events, SYNCHRONISES, and stores the best
 * GB/s (10^9 bytes/s) in *gbs. kind:
 *   EP_PROBE_READ   kernel reads `bytes` from src (device)            counts bytes
 *   EP_PROBE_WRITE  kernel writes `bytes` to dst (device)             counts bytes
 *   EP_PROBE_COPY   kernel copies src -> dst (device)                 counts 2*bytes
 *   EP_PROBE_MEMCPY cudaMemcpyAsync src -> dst, any direction         counts bytes
 * bytes must be a multiple of 16; buffers 16-byte aligned.
 */
#define EP_PROBE_READ   0
#define EP_PROBE_WRITE  1
#define EP_PROBE_COPY   2
#define EP_PROBE_MEMCPY 3
int ep_probe_bandwidth(int kind, void *dst, const void *src, size_t bytes, int iters, void *stream,
                       double *gbs);

/* Number of kernels this library has launched in this process (all threads). */
int64_t ep_launch_count(void);

const char *ep_strerror(int err);
/* cudaError_t value of the most recent failed CUDA call in this process, 0 if none. */
int ep_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* EP_B200_H */
