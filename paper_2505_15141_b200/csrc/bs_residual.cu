// bs_residual_sample: the resampling step of Algorithm 6 -- one token from Norm([P - Q]_+)
// at the first rejected position, or the bonus token from P when every draft passed.
// [.]_+ and Norm(.) as defined in the notation paragraph before Algorithm 6.
//
// One uniform per sequence, inverse CDF in vocabulary order.  Two levels, nobody waits:
//   level 1  a work item is one 32 KB segment of the (target, draft) row pair at position tau_b;
//            the CTA streams both rows with 128-bit loads, forms r_v = max(0, p_v - q_v) using
//            the row statistics left in the workspace by bs_softmax_verify, and writes the
//            segment mass.  An arrival counter per sequence elects the last CTA.
//   level 2  that CTA scans the segment masses in fp64, picks the segment in which the
//            cumulative mass crosses u * R, re-reads that one segment (an L2 hit) with each
//            thread owning a contiguous chunk, scans the chunk masses, and the single thread
//            whose chunk contains the crossing walks it element by element.
#include "bs_common.cuh"

namespace bs {

struct ResidParams {
    const void* target;
    const void* draft;
    const int32_t* tokens;
    const int32_t* gamma;
    const int32_t* accept_len;
    const float* u_resample;
    int32_t* out_tokens;
    int32_t* out_len;
    uint32_t* ticket;
    int32_t* status;
    const float2* row_stats;
    float* resid_partial;
    int B, Gmax, V, R, S;
    int nseg, seg;
    float c;
};

constexpr int kMaxSeg = 128;          // V <= 2^20 and segments of >= 8192 elements
constexpr int kRUnroll = 4;           // 128-bit loads in flight per thread and per row

// Mass of one element.  kt / kd fold the row max and normaliser: p = 2^(x*c + kt).
struct MassFn {
    float c, kt, kd;
    bool bonus;
    __device__ __forceinline__ float operator()(float xt, float xd) const {
        float pv = ex2(fmaf(xt, c, kt));
        if (bonus) return pv;
        float qv = ex2(fmaf(xd, c, kd));
        return fmaxf(0.f, pv - qv);
    }
};

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

// Sum of the masses of elements [e0, e0 + n) of the row pair, whole CTA.
template <typename T>
__device__ __forceinline__ float segment_mass(const T* tp, const T* dp, int e0, int n, const MassFn& f, float* s_red) {
    constexpr int kVec = Elem<T>::kVec;
    const int tid = threadIdx.x;
    const T* ts = tp + e0;
    const T* ds = f.bonus ? ts : dp + e0;
    const bool aligned = ((reinterpret_cast<uintptr_t>(ts) | reinterpret_cast<uintptr_t>(ds)) & 15) == 0;
    float acc = 0.f;
    int done = 0;
    if (aligned) {
        const int nv = n / kVec;
        const uint4* tv = reinterpret_cast<const uint4*>(ts);
        const uint4* dv = reinterpret_cast<const uint4*>(ds);
        for (int base = 0; base < nv; base += kThreads * kRUnroll) {
            uint4 a[kRUnroll], d[kRUnroll];
#pragma unroll
            for (int k = 0; k < kRUnroll; ++k) {
                int i = base + k * kThreads + tid;
                if (i < nv) {
                    a[k] = ld_stream(tv + i);
                    d[k] = f.bonus ? a[k] : ld_stream(dv + i);
                }
            }
#pragma unroll
            for (int k = 0; k < kRUnroll; ++k) {
                int i = base + k * kThreads + tid;
                if (i < nv) {
                    float ft[kVec], fd[kVec];
                    Elem<T>::unpack(a[k], ft);
                    Elem<T>::unpack(d[k], fd);
                    float s = 0.f;
#pragma unroll
                    for (int q = 0; q < kVec; ++q) s += f(ft[q], fd[q]);
                    acc += s;
                }
            }
        }
        done = nv * kVec;
    }
    for (int i = done + tid; i < n; i += kThreads)
        acc += f(Elem<T>::load(ts + i), f.bonus ? 0.f : Elem<T>::load(ds + i));
    return block_sum(acc, s_red);
}

template <typename T>
__global__ void __launch_bounds__(kThreads) residual_kernel(const ResidParams p) {
    __shared__ float s_red[kWarps];
    __shared__ double s_scan[kWarps];
    __shared__ double s_cum[kMaxSeg];
    __shared__ int s_flag;
    __shared__ int s_pick;
    __shared__ int s_token;
    __shared__ int s_lastpos;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int total = p.B * p.nseg;

    for (int item = blockIdx.x; item < total; item += gridDim.x) {
        const int b = item / p.nseg, sg = item - b * p.nseg;
        int g = p.gamma[b];
        if (g < 0 || g > p.Gmax) g = 0;
        int tau = p.accept_len[b];
        tau = max(0, min(tau, g));
        MassFn f;
        f.c = p.c;
        f.bonus = tau >= g;
        const float2 ts = p.row_stats[(size_t)b * p.R + tau];
        f.kt = -(ts.x * p.c + log2f(ts.y));
        f.kd = 0.f;
        const T* tp = row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, tau, p.V);
        const T* dp = tp;
        if (!f.bonus) {
            const float2 ds = p.row_stats[(size_t)b * p.R + p.Gmax + 1 + tau];
            f.kd = -(ds.x * p.c + log2f(ds.y));
            dp = row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, tau, p.V);
        }
        const int e0 = sg * p.seg;
        const int n = min(p.seg, p.V - e0);
        const float mass = segment_mass<T>(tp, dp, e0, n, f, s_red);
        if (tid == 0) {
            p.resid_partial[(size_t)b * p.S + sg] = mass;
            __threadfence();
            unsigned old = atomicAdd(p.ticket + b, 1u);
            s_flag = (old == (unsigned)(p.nseg - 1));
        }
        __syncthreads();
        if (s_flag) {
            // ---- last CTA of sequence b: inverse CDF ----
            __threadfence();
            int bits = 0;
            const float* pp = p.resid_partial + (size_t)b * p.S;
            if (tid == 0) {
                double cum = 0.0;
                for (int q = 0; q < p.nseg; ++q) { cum += (double)__ldcg(pp + q); s_cum[q] = cum; }
            }
            __syncthreads();
            double Rtot = s_cum[p.nseg - 1];
            if (!(Rtot > 0.0) || !isfinite(Rtot)) {
                // [P - Q]_+ has no mass (P == Q up to rounding) or the row is not finite:
                // fall back to the target distribution of the same row
                bits |= f.bonus ? BS_DEV_NONFINITE : BS_DEV_RESIDUAL_FALLBACK;
                f.bonus = true;
                __syncthreads();
                for (int q = 0; q < p.nseg; ++q) {
                    const int qe0 = q * p.seg;
                    float m2 = segment_mass<T>(tp, tp, qe0, min(p.seg, p.V - qe0), f, s_red);
                    if (tid == 0) s_cum[q] = (q ? s_cum[q - 1] : 0.0) + (double)m2;
                }
                __syncthreads();
                Rtot = s_cum[p.nseg - 1];
                if (!(Rtot > 0.0) || !isfinite(Rtot)) bits |= BS_DEV_NONFINITE;
            }
            const double target = (double)p.u_resample[b] * Rtot;
            if (tid == 0) {
                int pick = -1, lastpos = 0;
                for (int q = 0; q < p.nseg; ++q) {
                    if ((q ? s_cum[q] - s_cum[q - 1] : s_cum[0]) > 0.0) lastpos = q;
                    if (pick < 0 && s_cum[q] > target) pick = q;
                }
                s_pick = pick < 0 ? lastpos : pick;
                s_token = -1;
                s_lastpos = -1;
            }
            __syncthreads();
            const int ps = s_pick;
            const double t_in = target - (ps ? s_cum[ps - 1] : 0.0);
            // chunk of this thread inside the picked segment, in vocabulary order
            const int pe0 = ps * p.seg;
            const int pn = min(p.seg, p.V - pe0);
            const int chunk = div_up(pn, kThreads);
            const int c0 = min(pn, tid * chunk), c1 = min(pn, c0 + chunk);
            const T* ts2 = tp + pe0;
            const T* ds2 = dp + pe0;
            float csum = 0.f;
            int lastpos = -1;
            for (int i = c0; i < c1; ++i) {
                float r = f(Elem<T>::load(ts2 + i), f.bonus ? 0.f : Elem<T>::load(ds2 + i));
                csum += r;
                if (r > 0.f) lastpos = i;
            }
            // inclusive scan of the chunk masses over the CTA, fp64
            double incl = (double)csum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                double t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) s_scan[warp] = incl;
            __syncthreads();
            double woff = 0.0;
            for (int w = 0; w < warp; ++w) woff += s_scan[w];
            incl += woff;
            const double excl = incl - (double)csum;
            if (lastpos >= 0) atomicMax(&s_lastpos, lastpos);
            if (incl > t_in && !(excl > t_in)) {
                // the crossing lies in this chunk (exactly one thread satisfies both)
                double run = excl;
                int tok = -1;
                for (int i = c0; i < c1; ++i) {
                    float r = f(Elem<T>::load(ts2 + i), f.bonus ? 0.f : Elem<T>::load(ds2 + i));
                    run += (double)r;
                    if (run > t_in && r > 0.f) { tok = i; break; }
                }
                if (tok < 0) tok = lastpos;          // rounding between the two passes
                if (tok >= 0) s_token = pe0 + tok;
            }
            __syncthreads();
            if (tid == 0) {
                int tok = s_token;
                if (tok < 0) tok = (s_lastpos >= 0) ? pe0 + s_lastpos : 0;   // u * R beyond the recomputed mass
                int32_t* ot = p.out_tokens + (size_t)b * (p.Gmax + 1);
                for (int j = 0; j <= p.Gmax; ++j)
                    ot[j] = j < tau ? p.tokens[(size_t)b * p.Gmax + j] : (j == tau ? tok : -1);
                p.out_len[b] = tau + 1;
                if (bits) p.status[b] |= bits;
                p.ticket[b] = 0u;
            }
        }
        __syncthreads();
    }
}

// Greedy mode: the emitted token is the arg-max of target row tau, already in the row statistics.
__global__ void greedy_emit_kernel(const ResidParams p) {
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

static int g_rocc[2][64];

template <typename T>
static bs_status launch_residual(const ResidParams& p, int variant, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!g_rocc[variant][dev]) {
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, residual_kernel<T>, kThreads, 0) != cudaSuccess || occ < 1)
            occ = 1;
        g_rocc[variant][dev] = occ;
    }
    long long grid = (long long)sm_count() * g_rocc[variant][dev];
    const long long items = (long long)p.B * p.nseg;
    if (grid > items) grid = items;
    residual_kernel<T><<<(unsigned)grid, kThreads, 0, st>>>(p);
    return cuda_status(cudaGetLastError());
}

}  // namespace bs

using namespace bs;

extern "C" bs_status bs_residual_sample(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                        const int32_t* draft_tokens, const int32_t* gamma, const int32_t* accept_len,
                                        const float* u_resample, float temperature, int B, int Gmax, int V,
                                        int32_t* out_tokens, int32_t* out_len,
                                        void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 1 || Gmax < 0 || V < 1) return BS_ERR_INVALID_ARG;
    if (B > BS_MAX_BATCH || Gmax > BS_MAX_GAMMA || V > (1 << 20)) return BS_ERR_UNSUPPORTED;
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
    p.B = B; p.Gmax = Gmax; p.V = V; p.R = w.R; p.S = w.S;
    p.seg = seg_elems(dtype);
    p.nseg = div_up(V, p.seg);
    p.c = greedy ? 1.f : kLog2e / temperature;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (greedy) {
        greedy_emit_kernel<<<div_up(B, 128), 128, 0, st>>>(p);
        return cuda_status(cudaGetLastError());
    }
    return dtype == BS_F32 ? launch_residual<float>(p, 0, st) : launch_residual<__nv_bfloat16>(p, 1, st);
}
