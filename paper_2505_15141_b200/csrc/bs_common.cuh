// Shared device helpers and the workspace layout of the verification kernels.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <math.h>

#include "banditspec.h"

namespace bs {

constexpr int kThreads = 256;              // threads per CTA of the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kSegBytes = 32768;           // row-statistics kernels: bytes of one row segment = one work item
                                           // = one pipeline stage
constexpr int kSegElemsMin = kSegBytes / 4;  // segment length of the widest dtype (fp32)
constexpr int kResSegBytes = 16384;        // resampling kernel: bytes of one row segment
constexpr int kResSegElemsMin = kResSegBytes / 4;
constexpr int kResSubSegs = 16;            // pieces of a segment whose masses are kept separately (one per consumer warp)
constexpr float kLog2e = 1.4426950408889634f;

__host__ __device__ inline int seg_elems(int dtype) { return dtype == BS_F32 ? kSegBytes / 4 : kSegBytes / 2; }
__host__ __device__ inline int res_seg_elems(int dtype) { return dtype == BS_F32 ? kResSegBytes / 4 : kResSegBytes / 2; }
__host__ __device__ inline int div_up(int a, int b) { return (a + b - 1) / b; }
__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace regions (all offsets multiples of 256 bytes).
//   ticket_verify [B] u32     per-sequence arrival counters of the statistics kernel (zero between calls)
//   ticket_resid  [B] u32     per-sequence arrival counters of the resampling kernel (zero between calls)
//   ticket_row    [B, R] u32  first B words: bit j set = the statistics of draft row j were left by a
//                             drafting call (bs_draft_sample) and not yet consumed, bit 31 = a drafting pass
//                             met a row it could not sample; second B words: decision
//                             words of bs_verify_walk (zero between calls); rest unused
//   status        [B] i32     device-data status bits of the last call pair
//   abort         [1] i32     set when a bounded pipeline wait gave up (reported as BS_ERR_TIMEOUT)
//   row_stats     [B, R, 2] f32, R = 2*Gmax+1: (raw max logit, Z) per row; greedy: (max, arg-max bits)
//                 rows 0..Gmax are target rows, rows Gmax+1..2*Gmax are draft rows
//   partial       [B, R, S, 2] f32, S = ceil(V / 8192): per-segment (max, Z) / (max, arg-max)
//   resid_partial [B, Sr] f32, Sr = 16 * ceil(V / 4096): residual mass of every 1 KB piece of a row pair
//                 (the generic kernel uses one entry per 16 KB segment)
struct Workspace {
    size_t off_ticket_verify, off_ticket_resid, off_ticket_row, off_status, off_abort, off_row_stats, off_partial,
        off_resid_partial, total;
    int R, S, Sr;
};

__host__ __device__ inline Workspace workspace_layout(int B, int Gmax, int V) {
    Workspace w;
    w.R = 2 * Gmax + 1;
    w.S = div_up(V, kSegElemsMin);
    w.Sr = kResSubSegs * div_up(V, kResSegElemsMin);
    size_t o = 0;
    w.off_ticket_verify = o; o = align_up(o + sizeof(uint32_t) * (size_t)B, 256);
    w.off_ticket_resid = o;  o = align_up(o + sizeof(uint32_t) * (size_t)B, 256);
    w.off_ticket_row = o;    o = align_up(o + sizeof(uint32_t) * (size_t)B * (w.R < 2 ? 2 : w.R), 256);
    w.off_status = o;        o = align_up(o + sizeof(int32_t) * (size_t)B, 256);
    w.off_abort = o;         o = align_up(o + sizeof(int32_t), 256);
    w.off_row_stats = o;     o = align_up(o + sizeof(float) * 2 * (size_t)B * w.R, 256);
    w.off_partial = o;       o = align_up(o + sizeof(float) * 2 * (size_t)B * w.R * w.S, 256);
    w.off_resid_partial = o; o = align_up(o + sizeof(float) * (size_t)B * w.Sr, 256);
    w.total = o;
    return w;
}

// ---- small device helpers -----------------------------------------------------------

__device__ __forceinline__ float ex2(float x) {           // 2^x, MUFU
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {   // read-once 128-bit load
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;                           // elements per 128-bit load
    static constexpr int kDtype = BS_F32;
    __device__ static __forceinline__ float load(const float* p) { return __ldg(p); }
    __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    static constexpr int kDtype = BS_BF16;
    __device__ static __forceinline__ float load(const __nv_bfloat16* p) {
        return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float* f) {   // bf16 -> fp32 is a shift
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};

// Row r of sequence b in the [B, rows_per_seq, V] tensor.
template <typename T>
__device__ __forceinline__ const T* row_ptr(const T* base, int b, int rows_per_seq, int r, int V) {
    return base + ((size_t)b * rows_per_seq + r) * (size_t)V;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// (m, s) pairs of an online softmax: s = sum exp2((x - m) * c).  Merging rescales to the larger m.
__device__ __forceinline__ float rescale(float m_from, float m_to, float c) {
    // factor that takes a sum expressed relative to m_from to one relative to m_to (m_to >= m_from)
    return (m_from == -INFINITY) ? 0.f : ex2((m_from - m_to) * c);
}

extern thread_local int g_last_cuda_error;      // last failing cudaError_t seen by this thread (diagnostics only)
inline bs_status cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return BS_OK;
    g_last_cuda_error = (int)e;
    cudaGetLastError();                          // clear the sticky launch error
    return BS_ERR_CUDA;
}

int sm_count();            // SMs of the current device (cached per device)

// Programmatic dependent launch.  Every kernel of the library is launched with the attribute that
// lets it start while the kernel before it on the stream is still draining: its CTAs take SMs as
// they free up and run whatever does not touch global memory (barrier set-up, tensor-memory
// allocation); pdl_wait() then holds them until the earlier grid has completed and its writes are
// visible, and only after that pdl_release() lets the kernel behind this one do the same, so at
// most two grids overlap.  Without the attribute both calls do nothing.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_wait(); pdl_release(); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
#ifdef BS_NO_PDL                                   // build-time switch for A/B timing: plain stream order
    cfg.numAttrs = 0;
#endif
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

}  // namespace bs
