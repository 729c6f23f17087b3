// Device helpers shared by the layout kernels: divisions by launch-time constants as high
// multiplies, and an exclusive scan over a shared-memory array.
#pragma once

#include "ep_common.cuh"

namespace ep {

// n / d for 0 <= n < 2^31 by one 64x64 high multiply: m = ceil(2^64 / d)
struct FastDiv {
    uint32_t d;
    uint64_t m;
};
inline FastDiv make_fastdiv(int d)
{
    FastDiv f;
    f.d = (uint32_t)d;
    f.m = d > 1 ? ~uint64_t(0) / (uint64_t)d + 1 : 0;
    return f;
}
__device__ __forceinline__ int fdiv(int n, const FastDiv &f)
{
    return f.d == 1 ? n : (int)__umul64hi((uint64_t)(uint32_t)n, f.m);
}
// n / d by one 32-bit high multiply with mul = ceil(2^32 / d) (0 stands for d == 1): exact while
// n * d < 2^32, which holds for an expert id over E/R (both <= 4096) and a pair index of a group over K.
inline uint32_t small_div_mul(int d) { return d > 1 ? 0xffffffffu / (uint32_t)d + 1u : 0u; }
__device__ __forceinline__ int sdiv(int n, uint32_t mul) { return mul ? (int)__umulhi((uint32_t)n, mul) : n; }

#ifdef __CUDACC__
// Sums of one counter over the CTAs' scratch rows: col[c * stride] over c in [0, n) and over c in [0, n_before), kBatch
// loads (L2, written by another kernel) requested before the first is used. `never` is a launch argument that the host
// has checked to be false; the compiler cannot know, so the store behind it (never executed) ends the basic block between
// the requests and the sums. Inside one block the compiler hands the batch's loads to the warp's six scoreboards group
// after group and the thread pays an L2 round trip per group: with the block split the pair half of the layout of 8192
// tokens takes 9.5 us per call instead of 10.5 (12.0 with a plainly unrolled loop).
template <int kBatch>
__device__ __forceinline__ void column_sums(const int32_t *col, size_t stride, int n, int n_before, bool never, int32_t *sink,
                                            int32_t *total_out, int32_t *before_out)
{
    int32_t total = 0, before = 0;
    for (int c0 = 0; c0 < n; c0 += kBatch) {
        int32_t v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) v[u] = __ldcg(col + (size_t)min(c0 + u, n - 1) * stride);   // past the end: the last row again
        if (never && threadIdx.x == 0) *sink = (int32_t)clock64();
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (c0 + u < n) total += v[u];
            if (c0 + u < n_before) before += v[u];
        }
    }
    *total_out = total;
    *before_out = before;
}

// exclusive scan of v[0..n) in place (shared memory), v[n] = total; whole CTA; sh holds one int per warp.
// Up to 1024 entries one warp does it alone (a chunk per lane, one shuffle scan, no block barrier inside).
static __device__ void block_exclusive_scan_smem(int32_t *v, int n, int32_t *sh)
{
    const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    if (n <= 1024) {
        if (warp == 0) {
            const int chunk = (n + 31) >> 5;
            const int lo = min(n, lane * chunk), hi = min(n, lo + chunk);
            int32_t sum = 0;
            for (int i = lo; i < hi; ++i) sum += v[i];
            int32_t incl = sum;
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t up = __shfl_up_sync(kFullMask, incl, off);
                if (lane >= off) incl += up;
            }
            int32_t run = incl - sum;
            for (int i = lo; i < hi; ++i) {
                const int32_t x = v[i];
                v[i] = run;
                run += x;
            }
            if (lane == 31) v[n] = incl;
        }
        __syncthreads();
        return;
    }
    const int chunk = (n + nt - 1) / nt;
    const int lo = min(n, tid * chunk), hi = min(n, lo + chunk);
    int32_t sum = 0;
    for (int i = lo; i < hi; ++i) sum += v[i];
    int32_t incl = sum;                              // inclusive scan of the chunk sums inside the warp
    for (int off = 1; off < 32; off <<= 1) {
        const int32_t up = __shfl_up_sync(kFullMask, incl, off);
        if (lane >= off) incl += up;
    }
    if (lane == 31) sh[warp] = incl;
    __syncthreads();
    if (warp == 0) {                                 // exclusive scan of the warp totals
        const int32_t w = lane < nw ? sh[lane] : 0;
        int32_t wi = w;
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t up = __shfl_up_sync(kFullMask, wi, off);
            if (lane >= off) wi += up;
        }
        if (lane < nw) sh[lane] = wi - w;
    }
    __syncthreads();
    int32_t run = sh[warp] + incl - sum;
    for (int i = lo; i < hi; ++i) {
        const int32_t x = v[i];
        v[i] = run;
        run += x;
    }
    if (tid == nt - 1) v[n] = run;
    __syncthreads();
}
#endif

}  // namespace ep
