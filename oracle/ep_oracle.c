/*
 * CPU oracle for routing-aware expert-parallel token dispatch and combine.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain statement of what the
 * path computes; the CUDA library shares no code with it and never calls it.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may build or
 * call it.
 *
 * What the paper fixes (Section 1, Section 2.1 "Distributed MoE and expert
 * parallelism" and "Communication patterns of dispatch and combine"; Section
 * 4.3; Section 4.5 "Routing-aware communication"): a router picks K of E experts
 * per token; experts are partitioned over R devices; every device owns a block of
 * tokens; dispatch sends a token's activation to each device that hosts one of
 * its picked experts -- only there, and once per device (the transfer volume
 * stops growing once a token reaches every device); each device groups what it
 * received by the experts it owns (a local permutation); combine returns the
 * expert outputs to the token's owner and sums them on the GPU in the
 * activation's arithmetic. The paper prints no algorithm, layout or number for
 * this path, so the definitions below are the plain set definitions of those
 * sentences under the following readings:
 *
 *   - token t belongs to source rank  t div (T/R)   (contiguous equal blocks)
 *   - expert e lives on rank          e div (E/R), local id e mod (E/R)
 *   - pair order: (t,k) before (t',k') iff t < t' or (t == t' and k < k');
 *     because source ranks own contiguous token blocks this is the order
 *     (source rank, token index, k)
 *   - an entry topk_idx[t][k] == -1 is masked: it is skipped everywhere; any
 *     other id outside [0,E) is skipped too and raises status bit 1
 *   - receive space: one row per distinct (token, destination rank), rows of a
 *     rank contiguous, ordered by token (hence by source rank, then token)
 *   - pair space: one entry per valid (t,k), grouped by global expert id (hence
 *     by rank, then local expert), ordered by (t,k) inside an expert
 *   - combine: fp32 fused multiply-add chain from +0 in ascending k, one
 *     round-to-nearest-even narrowing to bf16 at the end
 *
 * Pins (tests, CPU only). The paper prints no worked values for this path, so
 * every function here is pinned by the mathematics instead: brute-force
 * evaluation of the set expressions on tiny inputs; numpy bincount / cumsum /
 * stable argsort on every config; closed forms (R = 1, E = R, one-hot weights,
 * K = 1, constant rows); the invariants (counts sum to the number of valid
 * pairs; receive rows = number of distinct (token, rank); rows <= T*min(K,R);
 * identity expert with weights summing to 1 returns x); the constructed case of
 * the paper's Figure 3 caption; exact-rational evaluation of the combine chains
 * with explicit roundings; and, for the dense formulation, the paper's volume
 * formulas of Section 4.2.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_STATUS_BAD_INDEX 1

static float bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* round to nearest, ties to even; NaN stays NaN (quiet) */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u)
        return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/*
 * Layout. One sequential sweep over the pairs in (t,k) order with running
 * counters: the number of earlier pairs of the same expert, and the number of
 * earlier tokens that hit the same rank, are exactly what the counters hold when
 * the sweep reaches (t,k).
 *
 * Outputs (all int32, caller-allocated):
 *   expert_counts[E], expert_offsets[E+1], rank_rows[R], rank_row_offsets[R+1],
 *   src_row_offsets[R*(R+1)], recv_slot[T*K], pair_slot[T*K],
 *   recv_token[>= N_recv], pair_row[>= P], pair_token[>= P], status[1].
 * Returns 0, or -1 on a shape that the definitions do not cover.
 */
int ep_oracle_layout(int T, int K, int E, int R, const int32_t *topk_idx,
                     int32_t *expert_counts, int32_t *expert_offsets,
                     int32_t *rank_rows, int32_t *rank_row_offsets,
                     int32_t *src_row_offsets, int32_t *recv_slot,
                     int32_t *pair_slot, int32_t *recv_token, int32_t *pair_row,
                     int32_t *pair_token, int32_t *status)
{
    if (T < 0 || K < 1 || E < 1 || R < 1 || E % R != 0 || T % R != 0)
        return -1;
    const int El = E / R;       /* experts per rank */
    const int Tr = T / R;       /* tokens per source rank */
    int st = 0;

    /* counts */
    for (int e = 0; e < E; ++e) expert_counts[e] = 0;
    for (int r = 0; r < R; ++r) rank_rows[r] = 0;
    unsigned char *hit = (unsigned char *)calloc((size_t)(T > 0 ? T : 1) * R, 1);
    if (!hit) return -1;
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < K; ++k) {
            int e = topk_idx[(size_t)t * K + k];
            if (e == -1) continue;
            if (e < 0 || e >= E) { st |= ORACLE_STATUS_BAD_INDEX; continue; }
            expert_counts[e] += 1;
            hit[(size_t)t * R + e / El] = 1;
        }
    for (int t = 0; t < T; ++t)
        for (int r = 0; r < R; ++r)
            rank_rows[r] += hit[(size_t)t * R + r];

    /* exclusive prefix sums */
    expert_offsets[0] = 0;
    for (int e = 0; e < E; ++e) expert_offsets[e + 1] = expert_offsets[e] + expert_counts[e];
    rank_row_offsets[0] = 0;
    for (int r = 0; r < R; ++r) rank_row_offsets[r + 1] = rank_row_offsets[r] + rank_rows[r];

    /* sweep in (t,k) order */
    int32_t *seen_e = (int32_t *)calloc((size_t)E, sizeof(int32_t)); /* earlier pairs of expert e */
    int32_t *seen_r = (int32_t *)calloc((size_t)R, sizeof(int32_t)); /* earlier tokens hitting rank r */
    if (!seen_e || !seen_r) { free(hit); free(seen_e); free(seen_r); return -1; }
    for (int t = 0; t < T; ++t) {
        if (Tr > 0 && t % Tr == 0) {
            int s = t / Tr;     /* first token of source rank s */
            for (int r = 0; r < R; ++r)
                src_row_offsets[r * (R + 1) + s] = rank_row_offsets[r] + seen_r[r];
        }
        for (int k = 0; k < K; ++k) {
            size_t i = (size_t)t * K + k;
            int e = topk_idx[i];
            if (e < 0 || e >= E) { recv_slot[i] = -1; pair_slot[i] = -1; continue; }
            int r = e / El;
            int row = rank_row_offsets[r] + seen_r[r];   /* tokens t' < t with hit(t', r) */
            int p = expert_offsets[e] + seen_e[e];
            seen_e[e] += 1;
            recv_slot[i] = row;
            pair_slot[i] = p;
            recv_token[row] = t;
            pair_row[p] = row;
            pair_token[p] = t;
        }
        for (int r = 0; r < R; ++r) seen_r[r] += hit[(size_t)t * R + r];
    }
    for (int r = 0; r < R; ++r) {
        if (T == 0)
            for (int s = 0; s < R; ++s) src_row_offsets[r * (R + 1) + s] = 0;
        src_row_offsets[r * (R + 1) + R] = rank_row_offsets[r + 1];
    }
    *status = st;
    free(hit); free(seen_e); free(seen_r);
    return 0;
}

/*
 * Dispatch: recv[recv_slot[t][k]] = x[t], a bit copy of one bf16 row, for every
 * valid pair. Rows that no pair names are left untouched.
 */
int ep_oracle_dispatch(int T, int K, int H, const uint16_t *x, const int32_t *recv_slot,
                       uint16_t *recv, int64_t recv_rows)
{
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < K; ++k) {
            int32_t row = recv_slot[(size_t)t * K + k];
            if (row < 0) continue;
            if (row >= recv_rows) return -1;
            memcpy(recv + (size_t)row * H, x + (size_t)t * H, (size_t)H * sizeof(uint16_t));
        }
    return 0;
}

/*
 * Combine, as the path computes it: for each token and column an fp32 fused
 * multiply-add chain from +0 over k = 0..K-1 (masked slots skipped), then one
 * round-to-nearest-even narrowing to bf16.
 */
int ep_oracle_combine_f32(int T, int K, int H, const uint16_t *out, int64_t out_rows,
                          const int32_t *slot, const float *w, uint16_t *y)
{
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < H; ++h) {
            float acc = 0.0f;
            for (int k = 0; k < K; ++k) {
                int32_t row = slot[(size_t)t * K + k];
                if (row < 0) continue;
                if (row >= out_rows) return -1;
                acc = fmaf(w[(size_t)t * K + k], bf16_to_f32(out[(size_t)row * H + h]), acc);
            }
            y[(size_t)t * H + h] = f32_to_bf16_rne(acc);
        }
    return 0;
}

/*
 * Combine, the sum itself: y[t][h] = sum_k w[t][k] * out[slot[t][k]][h] in
 * fp64 (each product of an fp32 and a bf16 value is exact in fp64), not
 * narrowed. This is the reference of the tolerance test.
 */
int ep_oracle_combine_f64(int T, int K, int H, const uint16_t *out, int64_t out_rows,
                          const int32_t *slot, const float *w, double *y)
{
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                int32_t row = slot[(size_t)t * K + k];
                if (row < 0) continue;
                if (row >= out_rows) return -1;
                acc += (double)w[(size_t)t * K + k] * (double)bf16_to_f32(out[(size_t)row * H + h]);
            }
            y[(size_t)t * H + h] = acc;
        }
    return 0;
}

/* ------------------------------------------------------------------------
 * Variants around the path (Section 2.1, "Communication patterns of dispatch
 * and combine"; Section 4.3).
 * ------------------------------------------------------------------------ */

/*
 * Local grouping by expert (Section 4.3: each device groups the tokens it
 * received by the experts it owns): grouped[p] = recv[pair_row[p]].
 */
int ep_oracle_group(int64_t n_pairs, int H, const uint16_t *recv, int64_t recv_rows,
                    const int32_t *pair_row, uint16_t *grouped)
{
    for (int64_t p = 0; p < n_pairs; ++p) {
        if (pair_row[p] < 0 || pair_row[p] >= recv_rows) return -1;
        memcpy(grouped + (size_t)p * H, recv + (size_t)pair_row[p] * H, (size_t)H * sizeof(uint16_t));
    }
    return 0;
}

/*
 * Combine with partial outputs (Section 2.1: an All-to-Allv "transfers only the
 * tokens and partial outputs required"): every destination rank first sums, per
 * token it received, the weighted outputs of its own experts, and sends that one
 * row back; the owner adds the rows of the ranks the token reached.
 *   stage 1, for each receive row rho = recv_slot[t][k] (one per (t, rank)):
 *     partial[rho] = bf16( fp32 fma chain over the k' (ascending) of token t
 *                          with recv_slot[t][k'] == rho of w[t][k']*out[pair_slot[t][k']] )
 *   stage 2, for each token: y[t] = bf16( fp32 sum, from +0, of partial[rho] over
 *     the token's distinct receive rows in the order of their first k ).
 * partial has recv_rows rows; rows no token names are left untouched.
 */
int ep_oracle_combine_partial(int T, int K, int H, const uint16_t *out, int64_t out_rows,
                              const int32_t *pair_slot, const int32_t *recv_slot, const float *w,
                              uint16_t *partial, int64_t recv_rows, uint16_t *y)
{
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < H; ++h) {
            float total = 0.0f;
            for (int k = 0; k < K; ++k) {
                const int32_t rho = recv_slot[(size_t)t * K + k];
                if (rho < 0) continue;
                if (rho >= recv_rows) return -1;
                int first = 1;
                for (int k2 = 0; k2 < k; ++k2)
                    if (recv_slot[(size_t)t * K + k2] == rho) first = 0;
                if (!first) continue;
                float acc = 0.0f;                                   /* stage 1 on the expert's rank */
                for (int k2 = k; k2 < K; ++k2) {
                    if (recv_slot[(size_t)t * K + k2] != rho) continue;
                    const int32_t p = pair_slot[(size_t)t * K + k2];
                    if (p < 0 || p >= out_rows) return -1;
                    acc = fmaf(w[(size_t)t * K + k2], bf16_to_f32(out[(size_t)p * H + h]), acc);
                }
                const uint16_t sent = f32_to_bf16_rne(acc);          /* what travels back */
                partial[(size_t)rho * H + h] = sent;
                total = total + bf16_to_f32(sent);                   /* stage 2 on the owner */
            }
            y[(size_t)t * H + h] = f32_to_bf16_rne(total);
        }
    return 0;
}

/*
 * Dense formulation (Section 2.1: All-Gather and Reduce-Scatter; Figure 3).
 * Dispatch: every rank gathers the tokens of all ranks: gathered[r][t] = x[t],
 * R*T rows whatever the routing.
 */
int ep_oracle_dense_allgather(int T, int H, int R, const uint16_t *x, uint16_t *gathered)
{
    for (int r = 0; r < R; ++r)
        memcpy(gathered + (size_t)r * T * H, x, (size_t)T * H * sizeof(uint16_t));
    return 0;
}

/*
 * Dense combine: rank r places its partial outputs in a dense buffer ordered by
 * source token, dense[r][t] = bf16( fma chain over the k (ascending) whose expert
 * lives on r ), +0 where the token has no expert on r; the reduce-scatter returns
 * y[t] = bf16( fp32 sum from +0 over r = 0..R-1 of dense[r][t] ) to the owner.
 */
int ep_oracle_dense_reduce_scatter(int T, int K, int H, int E, int R, const int32_t *topk_idx,
                                   const uint16_t *out, int64_t out_rows, const int32_t *pair_slot,
                                   const float *w, uint16_t *dense, uint16_t *y)
{
    if (E % R != 0) return -1;
    const int El = E / R;
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < H; ++h) {
            float total = 0.0f;
            for (int r = 0; r < R; ++r) {
                float acc = 0.0f;
                for (int k = 0; k < K; ++k) {
                    const int e = topk_idx[(size_t)t * K + k];
                    if (e < 0 || e >= E || e / El != r) continue;
                    const int32_t p = pair_slot[(size_t)t * K + k];
                    if (p < 0 || p >= out_rows) return -1;
                    acc = fmaf(w[(size_t)t * K + k], bf16_to_f32(out[(size_t)p * H + h]), acc);
                }
                const uint16_t placed = f32_to_bf16_rne(acc);
                dense[((size_t)r * T + t) * H + h] = placed;
                total = total + bf16_to_f32(placed);
            }
            y[(size_t)t * H + h] = f32_to_bf16_rne(total);
        }
    return 0;
}
