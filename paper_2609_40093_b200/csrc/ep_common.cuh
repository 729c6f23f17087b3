// Shared host/device helpers of the EP library: error plumbing, shape checks,
// 16-byte vector loads/stores with cache hints, bf16 <-> fp32 bit moves.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <mutex>

#include "../../include/ep.h"

namespace ep {

constexpr int kMaxTopK = 32;
constexpr int kMaxRanks = 64;
constexpr int kMaxExperts = 4096;
constexpr unsigned kFullMask = 0xffffffffu;

// --- host side ------------------------------------------------------------

void note_cuda_error(cudaError_t e);       // remembers the code for ep_last_cuda_error
void count_launches(int n);                // feeds ep_launch_count

// Ordering events of the multi-stream entry points: *pool gets at least `need` timing-free events of
// the current device; `hold` owns the pool's mutex until the caller lets go of it (after its last
// record/wait has been enqueued). At most kOrderEventPool events per call.
constexpr int kOrderEventPool = 4352;   // 64*64 segments plus per-rank and per-call events
int order_events(cudaEvent_t **pool, int need, std::unique_lock<std::mutex> &hold);

#define EP_CUDA_TRY(expr)                                   \
    do {                                                    \
        cudaError_t _e = (expr);                            \
        if (_e != cudaSuccess) {                            \
            ::ep::note_cuda_error(_e);                      \
            return EP_ERR_CUDA;                             \
        }                                                   \
    } while (0)

// after a kernel launch: pick up launch-configuration errors without synchronising
#define EP_LAUNCH_CHECK(n_launched)                         \
    do {                                                    \
        ::ep::count_launches(n_launched);                   \
        EP_CUDA_TRY(cudaGetLastError());                    \
    } while (0)

// Would ep_layout run this call on its lean kernels (ep_layout.cu)? Then the layout followed by a dependent dispatch
// launch is faster than the one-launch form of ep_layout_dispatch at every batch size.
bool layout_is_lean(const ep_shape_t &shape, const void *topk_idx, const ep_layout_t &out, size_t workspace_bytes);

// Kernel launchers shared between the translation units (arguments already validated).
int launch_dispatch(const ep_shape_t &s, const void *x, const int32_t *recv_slot, void *recv,
                    int64_t capacity_rows, int32_t *status, cudaStream_t stream, bool behind_layout = false);
int launch_group(const ep_shape_t &s, const void *recv, int64_t recv_rows, const int32_t *pair_row,
                 const int32_t *n_pairs, void *grouped, int64_t capacity_rows, int32_t *status,
                 cudaStream_t stream);
int launch_combine(const ep_shape_t &s, const void *out, int64_t out_rows, const int32_t *slot,
                   const float *weights, void *y, int32_t *status, cudaStream_t stream);
int launch_permute(int hidden, const void *src, int64_t src_rows, const int32_t *src_slot, void *dst,
                   int64_t dst_rows, const int32_t *dst_slot, int64_t n, int32_t *status, cudaStream_t stream);
int launch_partial_rows(const ep_shape_t &s, const void *out, int64_t out_rows, const int32_t *pair_slot,
                        const int32_t *key, int dense, const float *weights, void *partial, int64_t partial_rows,
                        int32_t *status, cudaStream_t stream);
int launch_sum_partial_rows(int hidden, int top_k, const void *partial, int64_t partial_rows, const int32_t *slot,
                            void *y, int n_tokens, int32_t *status, cudaStream_t stream);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shape limits shared by every entry point. need_hidden: the call moves rows.
inline int check_shape(const ep_shape_t *s, bool need_hidden)
{
    if (!s) return EP_ERR_NULL;
    const int64_t T = s->num_tokens, K = s->top_k, H = s->hidden, E = s->num_experts, R = s->num_ranks;
    if (T < 0 || K < 1 || K > kMaxTopK || R < 1 || R > kMaxRanks) return EP_ERR_INVALID_ARG;
    if (E < R || E > kMaxExperts || E % R != 0 || T % R != 0) return EP_ERR_INVALID_ARG;
    if (T * K >= (int64_t(1) << 31)) return EP_ERR_INVALID_ARG;
    if (need_hidden && (H < 8 || H % 8 != 0)) return EP_ERR_INVALID_ARG;
    return EP_OK;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Launch through cudaLaunchKernelEx. pdl: with programmatic stream serialisation, i.e. the kernel's CTAs
// may become resident while the previous kernel of the stream is still running; the kernel must execute
// pdl_wait() before it touches anything an earlier kernel wrote. Stream order is otherwise unchanged.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args)
{
    return launch_kernel(true, kernel, grid, block, smem, stream, args...);
}

// --- device side ----------------------------------------------------------

#ifdef __CUDACC__

// Blocks until every kernel this one depends on has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream become resident (it still waits in its own pdl_wait()).
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ unsigned lanemask_lt()
{
    unsigned m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// Read-once 16-byte load: read-only path, do not keep the line in L1.
__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Write-once 16-byte store (streaming: evict first).
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// two fp32 -> packed bf16x2 (lo in bits 0..15), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

#endif  // __CUDACC__

}  // namespace ep
