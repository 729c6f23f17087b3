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
 * allocates device memory, prints, throws or aborts. Unless stated otherwise a
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
 *     bytes while the batch fits one thread-block cluster (2048 tokens, fewer
 *     when large E or K shrink the CTA), else 4*(E+R+1) bytes per CTA, at most
 *     128 CTAs (34 KB for T=8192, E=256, R=8). Shapes
 *     that need more than the array holds return EP_ERR_STATIC_SCRATCH and
 *     enqueue nothing.
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
 * Host-staged round trip with separate upload and download streams (Section
 * 4.3: uploads and downloads are issued on two different streams and cut into
 * chunks so that both directions of the host link are busy; Section 4.4: two alternating bounce
 * buffers). Packs the receive rows into `staging` (device) with the dispatch
 * kernel on stream_up, copies them chunk by chunk to the bounce buffer
 * (pinned host, 2 * staging_capacity_rows rows: half `round & 1` is used) and
 * from there into `recv` (device, same row layout) on stream_down. Each rank's
 * partition is cut into chunks_per_rank chunks. duplex != 0: a chunk's download
 * is released by an event right after its upload, so uploads and downloads
 * overlap; duplex == 0: all uploads, then all downloads. The result is complete
 * when stream_down is; stream_up first waits for what is queued on stream_down.
 * rank_row_offsets_host (host, [R+1]) must hold the layout's offsets. Events are
 * created on first use and kept (no device memory is allocated).
 */
int ep_host_roundtrip(const ep_shape_t *shape, const void *x, const int32_t *recv_slot,
                      const int32_t *rank_row_offsets_host, void *staging, int64_t staging_capacity_rows,
                      void *bounce_host, int round, void *recv, int chunks_per_rank, int duplex,
                      int32_t *status, void *stream_up, void *stream_down);

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
 * (the call orders itself after the previous one). 1 <= chunks <= 256.
 */
int ep_host_step_pipelined(const ep_shape_t *shape, const void *x_host, const int32_t *topk_idx_host,
                           const float *topk_weights_host, void *y_host, int32_t *status_host, void *arena,
                           size_t arena_bytes, int chunks, void *stream_in, void *stream_compute,
                           void *stream_out);

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
