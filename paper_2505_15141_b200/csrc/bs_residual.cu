// bs_residual_sample: the resampling step of Algorithm 6 -- one token from Norm([P - Q]_+)
// at the first rejected position, or the bonus token from P when every draft passed.
// [.]_+ and Norm(.) as defined in the notation paragraph before Algorithm 6.
//
// One uniform per sequence, inverse CDF in vocabulary order.  Two levels, nobody waits:
//   level 1  each sequence's (target, draft) row pair at position tau_b is split into 16 KB
//            segments, shared out contiguously over a few CTAs; a CTA streams its segments with
//            128-bit loads, forms r_v = max(0, p_v - q_v) using the row statistics left in the
//            workspace by bs_softmax_verify, and writes one mass per segment (no CTA-wide
//            synchronisation between segments).  An arrival counter per sequence elects the last CTA.
//   level 2  that CTA scans the segment masses in fp64 (one per thread), picks the segment in
//            which the cumulative mass crosses u * R, re-reads that one segment (an L2 hit) into
//            registers in the same coalesced layout, scans the per-vector masses across the CTA
//            in fp64, and the one thread whose vector contains the crossing walks its 4 or 8
//            elements.  The same r_v values feed the scan and the walk.
#include "bs_residual_common.cuh"

#include <limits.h>

namespace bs {

constexpr int kMaxSeg = BS_MAX_VOCAB / kResSegElemsMin;       // 256 = kThreads: one segment mass per thread
constexpr int kVecTrip = kResSegBytes / 16 / kThreads;        // 128-bit vectors per thread and row in one segment
static_assert(kMaxSeg <= kThreads, "level 2 scans one segment mass per thread");

// Masses of this thread's vectors of segment [e0, e0 + n): vector k covers elements
// (k * kThreads + tid) * kVec .. + kVec of the segment; elements past n get mass 0.
template <typename T>
__device__ __forceinline__ void segment_masses(const T* tp, const T* dp, int e0, int n, const MassFn& f,
                                               float (&r)[kVecTrip][Elem<T>::kVec]) {
    constexpr int kVec = Elem<T>::kVec;
    const int tid = threadIdx.x;
    const T* ts = tp + e0;
    const T* ds = f.bonus ? ts : dp + e0;
    const bool aligned = ((reinterpret_cast<uintptr_t>(ts) | reinterpret_cast<uintptr_t>(ds)) & 15) == 0;
    if (aligned) {
        uint4 a[kVecTrip], d[kVecTrip];
#pragma unroll
        for (int k = 0; k < kVecTrip; ++k) {
            const int e = (k * kThreads + tid) * kVec;
            if (e + kVec <= n) {
                a[k] = ld_stream(reinterpret_cast<const uint4*>(ts + e));
                d[k] = f.bonus ? a[k] : ld_stream(reinterpret_cast<const uint4*>(ds + e));
            }
        }
#pragma unroll
        for (int k = 0; k < kVecTrip; ++k) {
            const int e = (k * kThreads + tid) * kVec;
            if (e + kVec <= n) {
                float ft[kVec], fd[kVec];
                Elem<T>::unpack(a[k], ft);
                Elem<T>::unpack(d[k], fd);
#pragma unroll
                for (int q = 0; q < kVec; ++q) r[k][q] = f(ft[q], fd[q]);
            } else {
#pragma unroll
                for (int q = 0; q < kVec; ++q)
                    r[k][q] = (e + q < n) ? f(Elem<T>::load(ts + e + q), f.bonus ? 0.f : Elem<T>::load(ds + e + q)) : 0.f;
            }
        }
    } else {
#pragma unroll
        for (int k = 0; k < kVecTrip; ++k) {
            const int e = (k * kThreads + tid) * kVec;
#pragma unroll
            for (int q = 0; q < kVec; ++q)
                r[k][q] = (e + q < n) ? f(Elem<T>::load(ts + e + q), f.bonus ? 0.f : Elem<T>::load(ds + e + q)) : 0.f;
        }
    }
}

__device__ __forceinline__ float block_sum(float v, float* s_red) {   // fixed order; result in all threads
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += s_red[w];
    return t;
}

// Sum of this thread's masses of segment [e0, e0 + n).
template <typename T>
__device__ __forceinline__ float thread_mass(const T* tp, const T* dp, int e0, int n, const MassFn& f) {
    constexpr int kVec = Elem<T>::kVec;
    float r[kVecTrip][kVec];
    segment_masses<T>(tp, dp, e0, n, f, r);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < kVecTrip; ++k) {
        float s = 0.f;
#pragma unroll
        for (int q = 0; q < kVec; ++q) s += r[k][q];
        acc += s;
    }
    return acc;
}

// Inclusive scan over the CTA in thread order, fp64.  Returns this thread's inclusive value; `excl`
// gets the value of the thread before it (0 for thread 0) and `total` the sum over the CTA.
__device__ __forceinline__ double block_scan(double v, double* s_w, double& excl, double& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    double prev = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane == 0) prev = 0.0;
    __syncthreads();
    if (lane == 31) s_w[warp] = incl;
    __syncthreads();
    double woff = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        if (w == warp) woff = tot;
        tot += s_w[w];
    }
    total = tot;
    excl = woff + prev;
    return woff + incl;
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 2) residual_kernel(const ResidParams p, const int nsplit) {
    constexpr int kVec = Elem<T>::kVec;
    __shared__ float s_red[kWarps];
    __shared__ double s_w[kWarps];
    __shared__ float s_mass[kMaxSeg];
    __shared__ float s_wm[kMaxSeg][kWarps];
    __shared__ int s_flag;
    __shared__ int s_pick;
    __shared__ int s_lastseg;
    __shared__ int s_token;
    __shared__ int s_lastpos;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_enter();
    // CTA (b, part) owns a contiguous range of the segments of sequence b
    {
        const int b = blockIdx.x / nsplit, part = blockIdx.x - b * nsplit;
        const int sg0 = (int)((long long)p.nseg * part / nsplit);
        const int sg1 = (int)((long long)p.nseg * (part + 1) / nsplit);
        int g = p.gamma[b];
        if (g < 0 || g > p.Gmax) g = 0;
        const int tau = max(0, min(p.accept_len[b], g));
        MassFn f;
        f.c = p.c;
        f.bonus = tau >= g;
        const float2 ts = p.row_stats[(size_t)b * p.R + tau];
        MassFn::fold(ts.x, ts.y, p.c, f.kt, f.at);
        f.kd = 0.f; f.ad = 1.f;
        const T* tp = row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, tau, p.V);
        const T* dp = tp;
        if (!f.bonus) {
            const float2 ds = p.row_stats[(size_t)b * p.R + p.Gmax + 1 + tau];
            MassFn::fold(ds.x, ds.y, p.c, f.kd, f.ad);
            dp = row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, tau, p.V);
        }
        // ---- level 1: segment masses, no CTA-wide synchronisation between segments ----
        for (int sg = sg0; sg < sg1; ++sg) {
            const int e0 = sg * p.seg;
            const float w = warp_sum(thread_mass<T>(tp, dp, e0, min(p.seg, p.V - e0), f));
            if (lane == 0) s_wm[sg - sg0][warp] = w;
        }
        __syncthreads();
        if (tid < sg1 - sg0) {
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) t += s_wm[tid][w];         // fixed order
            p.resid_partial[(size_t)b * p.S + sg0 + tid] = t;
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned old = atomicAdd(p.ticket + b, 1u);
            s_flag = (old == (unsigned)(nsplit - 1));
        }
        __syncthreads();
        if (s_flag) {
            // ---- level 2, last CTA of sequence b: inverse CDF over the vocabulary ----
            __threadfence();
            int bits = 0;
            s_mass[tid] = tid < p.nseg ? __ldcg(p.resid_partial + (size_t)b * p.S + tid) : 0.f;
            double excl, Rtot;
            double incl = block_scan((double)s_mass[tid], s_w, excl, Rtot);
            if (!(Rtot > (f.bonus ? 0.0 : kResidualFloor)) || !isfinite(Rtot)) {
                // [P - Q]_+ has no mass (P == Q up to rounding) or the row is not finite:
                // fall back to the target distribution of the same row
                bits |= f.bonus ? BS_DEV_NONFINITE : BS_DEV_RESIDUAL_FALLBACK;
                f.bonus = true;
                for (int q = 0; q < p.nseg; ++q) {
                    const int qe0 = q * p.seg;
                    const float m2 = block_sum(thread_mass<T>(tp, tp, qe0, min(p.seg, p.V - qe0), f), s_red);
                    if (tid == q) s_mass[q] = m2;
                }
                __syncthreads();
                incl = block_scan((double)s_mass[tid], s_w, excl, Rtot);
                if (!(Rtot > 0.0) || !isfinite(Rtot)) bits |= BS_DEV_NONFINITE;
            }
            const double target = (double)p.u_resample[b] * Rtot;
            if (tid == 0) { s_pick = -1; s_lastseg = 0; s_token = INT_MAX; s_lastpos = -1; }
            __syncthreads();
            if (tid < p.nseg) {
                if (s_mass[tid] > 0.f) atomicMax(&s_lastseg, tid);
                if (incl > target && !(excl > target)) s_pick = tid;       // at most one thread
            }
            __syncthreads();
            const int ps = s_pick >= 0 ? s_pick : s_lastseg;
            // cumulative mass before the picked segment
            const double before = __shfl_sync(0xffffffffu, excl, ps & 31);     // valid in warp ps / 32
            if ((tid >> 5) == (ps >> 5) && (tid & 31) == 0) s_w[0] = before;
            __syncthreads();
            const double t_in = target - s_w[0];
            __syncthreads();
            // ---- inside the picked segment ----
            const int pe0 = ps * p.seg;
            const int pn = min(p.seg, p.V - pe0);
            float r[kVecTrip][kVec];
            segment_masses<T>(tp, dp, pe0, pn, f, r);
            double base = 0.0;
#pragma unroll
            for (int k = 0; k < kVecTrip; ++k) {
                float vs = 0.f;
                int lastq = -1;
#pragma unroll
                for (int q = 0; q < kVec; ++q) { vs += r[k][q]; if (r[k][q] > 0.f) lastq = q; }
                double vex, vtot;
                const double vin = base + block_scan((double)vs, s_w, vex, vtot);
                vex += base;
                const int e = (k * kThreads + tid) * kVec;
                if (lastq >= 0) atomicMax(&s_lastpos, e + lastq);
                if (vin > t_in && !(vex > t_in)) {
                    double run = vex;
                    int tok = -1;
#pragma unroll
                    for (int q = 0; q < kVec; ++q) {
                        run += (double)r[k][q];
                        if (tok < 0 && run > t_in && r[k][q] > 0.f) tok = q;
                    }
                    if (tok < 0) tok = lastq;
                    if (tok >= 0) atomicMin(&s_token, pe0 + e + tok);
                }
                base += vtot;
            }
            __syncthreads();
            if (tid == 0) {
                int tok = s_token;
                if (tok == INT_MAX) {                    // u * R at or beyond the recomputed mass of the segment
                    if (s_lastpos >= 0) tok = pe0 + s_lastpos;
                    else { tok = 0; bits |= BS_DEV_NONFINITE; }
                }
                int32_t* ot = p.out_tokens + (size_t)b * (p.Gmax + 1);
                for (int j = 0; j <= p.Gmax; ++j)
                    ot[j] = j < tau ? p.tokens[(size_t)b * p.Gmax + j] : (j == tau ? tok : -1);
                p.out_len[b] = tau + 1;
                if (bits) p.status[b] |= bits;
                p.ticket[b] = 0u;
            }
        }
    }
}

// Greedy mode: the emitted token is the arg-max of target row tau, already in the row statistics.
__global__ void greedy_emit_kernel(const ResidParams p) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= p.B) return;
    int g = p.gamma[b];
    if (g < 0 || g > p.Gmax) g = 0;
    const int tau = max(0, min(p.accept_len[b], g));
    const int tok = __float_as_int(p.row_stats[(size_t)b * p.R + tau].y);
    int32_t* ot = p.out_tokens + (size_t)b * (p.Gmax + 1);
    for (int j = 0; j <= p.Gmax; ++j)
        ot[j] = j < tau ? p.tokens[(size_t)b * p.Gmax + j] : (j == tau ? tok : -1);
    p.out_len[b] = tau + 1;
}

template <typename T>
static bs_status launch_residual(const ResidParams& p, cudaStream_t st) {
    // at most two CTAs per SM in total (one wave), each owning a contiguous share of one sequence's segments
    int nsplit = 2 * sm_count() / p.B;
    if (nsplit > p.nseg) nsplit = p.nseg;
    if (nsplit < 1) nsplit = 1;
    return cuda_status(launch_pdl(residual_kernel<T>, (unsigned)(p.B * nsplit), kThreads, 0, st, p, nsplit));
}

}  // namespace bs

using namespace bs;

extern "C" bs_status bs_residual_sample(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                        const int32_t* draft_tokens, const int32_t* gamma, const int32_t* accept_len,
                                        const float* u_resample, float temperature, int B, int Gmax, int V,
                                        int32_t* out_tokens, int32_t* out_len,
                                        void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 1 || Gmax < 0 || V < 1) return BS_ERR_INVALID_ARG;
    if (B > BS_MAX_BATCH || Gmax > BS_MAX_GAMMA || V > BS_MAX_VOCAB) return BS_ERR_UNSUPPORTED;
    if (dtype != BS_F32 && dtype != BS_BF16) return BS_ERR_INVALID_ARG;
    if (!(temperature >= 0.f) || !isfinite(temperature)) return BS_ERR_INVALID_ARG;
    const bool greedy = temperature == 0.f;
    if (!target_logits || !gamma || !accept_len || !out_tokens || !out_len || !workspace) return BS_ERR_INVALID_ARG;
    if (Gmax > 0 && !draft_tokens) return BS_ERR_INVALID_ARG;
    if (!greedy && (!u_resample || (Gmax > 0 && !draft_logits))) return BS_ERR_INVALID_ARG;
    const Workspace w = workspace_layout(B, Gmax, V);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) return BS_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    ResidParams p;
    p.target = target_logits; p.draft = draft_logits; p.tokens = draft_tokens; p.gamma = gamma;
    p.accept_len = accept_len; p.u_resample = u_resample; p.out_tokens = out_tokens; p.out_len = out_len;
    p.ticket = reinterpret_cast<uint32_t*>(ws + w.off_ticket_resid);
    p.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    p.row_stats = reinterpret_cast<const float2*>(ws + w.off_row_stats);
    p.resid_partial = reinterpret_cast<float*>(ws + w.off_resid_partial);
    p.abort_flag = reinterpret_cast<int32_t*>(ws + w.off_abort);
    p.B = B; p.Gmax = Gmax; p.V = V; p.R = w.R; p.S = w.Sr;
    p.seg = res_seg_elems(dtype);
    p.nseg = div_up(V, p.seg);
    p.c = greedy ? 1.f : kLog2e / temperature;
    p.mode = kResidVerify; p.position = 0; p.draft_out = nullptr; p.draft_ready = nullptr;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (greedy) {
        return cuda_status(launch_pdl(greedy_emit_kernel, div_up(B, 128), 128, 0, st, p));
    }
    // rows on 16-byte boundaries: bulk-copy pipeline; otherwise the generic kernel
    const size_t es = dtype == BS_F32 ? 4 : 2;
    const bool aligned = ((size_t)V * es) % 16 == 0 && (reinterpret_cast<uintptr_t>(target_logits) & 15) == 0 &&
                         (reinterpret_cast<uintptr_t>(draft_logits) & 15) == 0;
    if (aligned)
        return dtype == BS_F32 ? launch_residual_stream<float>(p, st) : launch_residual_stream<__nv_bfloat16>(p, st);
    return dtype == BS_F32 ? launch_residual<float>(p, st) : launch_residual<__nv_bfloat16>(p, st);
}

// Sampling pass of bs_draft_sample: the resampling kernel in its drafting mode, on the draft row
// `position` whose statistics the statistics pass has just left in the workspace.
bs_status bs::run_draft_resample(const void* draft_logits, bs_dtype dtype, int position, const int32_t* gamma,
                                 const float* u_draft, float temperature, int B, int Gmax, int V,
                                 int32_t* draft_tokens, void* workspace, size_t workspace_bytes, void* stream) {
    const Workspace w = workspace_layout(B, Gmax, V);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) return BS_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    ResidParams p;
    p.target = nullptr; p.draft = draft_logits; p.tokens = nullptr; p.gamma = gamma;
    p.accept_len = nullptr; p.u_resample = u_draft; p.out_tokens = nullptr; p.out_len = nullptr;
    p.ticket = reinterpret_cast<uint32_t*>(ws + w.off_ticket_resid);
    p.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    p.abort_flag = reinterpret_cast<int32_t*>(ws + w.off_abort);
    p.row_stats = reinterpret_cast<const float2*>(ws + w.off_row_stats);
    p.resid_partial = reinterpret_cast<float*>(ws + w.off_resid_partial);
    p.B = B; p.Gmax = Gmax; p.V = V; p.R = w.R; p.S = w.Sr;
    p.seg = res_seg_elems(dtype);
    p.nseg = div_up(V, p.seg);
    p.c = kLog2e / temperature;
    p.mode = kResidDraft; p.position = position; p.draft_out = draft_tokens;
    p.draft_ready = reinterpret_cast<uint32_t*>(ws + w.off_ticket_row);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return dtype == BS_F32 ? launch_residual_stream<float>(p, st) : launch_residual_stream<__nv_bfloat16>(p, st);
}
