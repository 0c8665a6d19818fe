// bs_softmax_verify: single-pass row softmax statistics over every valid target / draft row,
// then (by the last CTA to finish a sequence) token-probability gather, accept test and
// first-rejection scan.  Algorithm 6 of the paper, second line and for-loop; softmax with
// temperature as in Section 2.
//
// Work decomposition: a work item is one 32 KB segment of one valid row.  Sequences have
// ragged speculation lengths, so every CTA builds the prefix sum of items per sequence in
// shared memory and the persistent grid strides over the flat item list; rows beyond
// gamma_b cost nothing.  Each item is streamed with 128-bit read-once loads (8 in flight
// per thread), reduced to (max, sum exp) with ONE exp per logit, and written as a partial.
// An arrival counter per sequence (atomic ticket, nobody waits) elects the CTA that merges
// the partials and runs the accept scan.
#include "bs_common.cuh"

#include <limits.h>

namespace bs {

struct VerifyParams {
    const void* target;
    const void* draft;
    const int32_t* tokens;
    const int32_t* gamma;
    const float* u_accept;
    int32_t* accept_len;
    float* p_tok;
    float* q_tok;
    uint32_t* ticket;
    int32_t* status;
    float2* row_stats;
    float2* partial;
    int B, Gmax, V, R, S;
    int nseg, seg;     // segments per row and elements per segment for this dtype
    float c;           // log2(e) / temperature
};

constexpr int kUnroll = 8;      // 128-bit loads in flight per thread

struct ArgMax {
    float m;
    int idx;
};
__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b) {
    return (b.m > a.m || (b.m == a.m && b.idx < a.idx)) ? b : a;
}

// Running (m, s) of one thread: s = sum over seen x of exp2((x - m) * c).
struct Online {
    float m, s;
    __device__ __forceinline__ void raise_to(float mc, float c) {
        if (mc > m) { s *= rescale(m, mc, c); m = mc; }
    }
};

template <typename T>
__device__ __forceinline__ float chunk_max(const uint4 (&v)[kUnroll]);

template <>
__device__ __forceinline__ float chunk_max<float>(const uint4 (&v)[kUnroll]) {
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
        m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(v[k].x), __uint_as_float(v[k].y)),
                           fmaxf(__uint_as_float(v[k].z), __uint_as_float(v[k].w))));
    }
    return m;
}

template <>
__device__ __forceinline__ float chunk_max<__nv_bfloat16>(const uint4 (&v)[kUnroll]) {
    // packed max on the raw bf16 pairs: two elements per instruction
    __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&v[0].x);
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].x));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].y));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].z));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].w));
    }
    uint32_t w = *reinterpret_cast<uint32_t*>(&m2);
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

template <typename T> __device__ __forceinline__ uint4 neg_inf_vec();
template <> __device__ __forceinline__ uint4 neg_inf_vec<float>() {
    return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
}
template <> __device__ __forceinline__ uint4 neg_inf_vec<__nv_bfloat16>() {
    return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
}

// Items of sequence b: rows * segments.  An out-of-range gamma is processed as gamma = 0.
template <bool GREEDY>
__device__ __forceinline__ int seq_rows(int g, int Gmax) {
    if (g < 0 || g > Gmax) g = 0;
    return GREEDY ? g + 1 : 2 * g + 1;
}

template <typename T, bool GREEDY>
__global__ void __launch_bounds__(kThreads) verify_kernel(const VerifyParams p) {
    extern __shared__ int s_prefix[];            // [B + 1] exclusive prefix of items per sequence
    __shared__ float s_m[kWarps];
    __shared__ float s_s[kWarps];
    __shared__ int s_i[kWarps];
    __shared__ int s_flag;
    __shared__ float2 s_stats[2 * BS_MAX_GAMMA + 1];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kVec = Elem<T>::kVec;

    // ---- prefix sum of work items over the batch (every CTA, redundantly; B <= 4096) ----
    {
        const int per = div_up(p.B, kThreads);
        const int b0 = tid * per;
        int local = 0;
        for (int k = 0; k < per; ++k) {
            int b = b0 + k;
            if (b < p.B) local += seq_rows<GREEDY>(p.gamma[b], p.Gmax) * p.nseg;
        }
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_i[warp] = incl;
        __syncthreads();
        int woff = 0;
        for (int w = 0; w < warp; ++w) woff += s_i[w];
        int run = woff + incl - local;
        for (int k = 0; k < per; ++k) {
            int b = b0 + k;
            if (b < p.B) {
                s_prefix[b] = run;
                run += seq_rows<GREEDY>(p.gamma[b], p.Gmax) * p.nseg;
            }
        }
        if (tid == kThreads - 1) s_prefix[p.B] = run;     // last thread holds the grand total
        __syncthreads();
    }
    const int total = s_prefix[p.B];

    for (int item = blockIdx.x; item < total; item += gridDim.x) {
        // ---- locate (sequence, row, segment) ----
        int lo = 0, hi = p.B;                    // largest b with prefix[b] <= item
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (s_prefix[mid] <= item) lo = mid; else hi = mid;
        }
        const int b = lo;
        const int local = item - s_prefix[b];
        const int lr = local / p.nseg, sg = local - lr * p.nseg;
        int g = p.gamma[b];
        if (g < 0 || g > p.Gmax) g = 0;
        // local rows 0..g are target rows; g+1..2g are draft rows 0..g-1
        const bool is_target = lr <= g;
        const int r = is_target ? lr : p.Gmax + 1 + (lr - g - 1);
        const T* rowp = is_target
            ? row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, lr, p.V)
            : row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, lr - g - 1, p.V);
        const int e0 = sg * p.seg;
        const int n = min(p.seg, p.V - e0);
        const T* sp = rowp + e0;

        // split into scalar head (to the next 16-byte boundary), 128-bit body, scalar tail
        const int mis = (int)((reinterpret_cast<uintptr_t>(sp) & 15) / sizeof(T));
        const int head = mis ? min(n, kVec - mis) : 0;
        const int nv = (n - head) / kVec;
        const int tail0 = head + nv * kVec;
        const uint4* vp = reinterpret_cast<const uint4*>(sp + head);

        Online on{-INFINITY, 0.f};
        ArgMax am{-INFINITY, INT_MAX};

        if (tid < head) {
            float x = Elem<T>::load(sp + tid);
            if (GREEDY) { if (x > am.m) { am.m = x; am.idx = e0 + tid; } }
            else if (x != -INFINITY) { on.raise_to(x, p.c); on.s += ex2((x - on.m) * p.c); }
        }
        for (int base = 0; base < nv; base += kThreads * kUnroll) {
            uint4 v[kUnroll];
#pragma unroll
            for (int k = 0; k < kUnroll; ++k) {
                int i = base + k * kThreads + tid;
                v[k] = (i < nv) ? ld_stream(vp + i) : neg_inf_vec<T>();
            }
            if (GREEDY) {
#pragma unroll
                for (int k = 0; k < kUnroll; ++k) {
                    float f[kVec];
                    Elem<T>::unpack(v[k], f);
                    int ei = e0 + head + (base + k * kThreads + tid) * kVec;
#pragma unroll
                    for (int q = 0; q < kVec; ++q)
                        if (f[q] > am.m) { am.m = f[q]; am.idx = ei + q; }
                }
            } else {
                float mc = chunk_max<T>(v);
                on.raise_to(mc, p.c);
                if (on.m > -INFINITY) {
                    const float nm = -on.m * p.c;
                    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                    for (int k = 0; k < kUnroll; ++k) {
                        float f[kVec];
                        Elem<T>::unpack(v[k], f);
#pragma unroll
                        for (int q = 0; q < kVec; q += 2) {
                            acc0 += ex2(fmaf(f[q], p.c, nm));
                            acc1 += ex2(fmaf(f[q + 1], p.c, nm));
                        }
                    }
                    on.s += acc0 + acc1;
                }
            }
        }
        if (tid < n - tail0) {
            float x = Elem<T>::load(sp + tail0 + tid);
            if (GREEDY) { if (x > am.m) { am.m = x; am.idx = e0 + tail0 + tid; } }
            else if (x != -INFINITY) { on.raise_to(x, p.c); on.s += ex2((x - on.m) * p.c); }
        }

        // ---- block reduction (fixed order, deterministic) ----
        if (GREEDY) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                ArgMax t{__shfl_xor_sync(0xffffffffu, am.m, o), __shfl_xor_sync(0xffffffffu, am.idx, o)};
                am = better(am, t);
            }
            if (lane == 0) { s_m[warp] = am.m; s_i[warp] = am.idx; }
        } else {
            float wm = warp_max(on.m);
            float ws = warp_sum(on.s * rescale(on.m, wm, p.c));
            if (lane == 0) { s_m[warp] = wm; s_s[warp] = ws; }
        }
        __syncthreads();
        if (warp == 0) {
            float2 out;
            if (GREEDY) {
                ArgMax a{lane < kWarps ? s_m[lane] : -INFINITY, lane < kWarps ? s_i[lane] : INT_MAX};
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    ArgMax t{__shfl_xor_sync(0xffffffffu, a.m, o), __shfl_xor_sync(0xffffffffu, a.idx, o)};
                    a = better(a, t);
                }
                out = make_float2(a.m, __int_as_float(a.idx));
            } else {
                float m = lane < kWarps ? s_m[lane] : -INFINITY;
                float s = lane < kWarps ? s_s[lane] : 0.f;
                float M = warp_max(m);
                float Z = warp_sum(s * rescale(m, M, p.c));
                out = make_float2(M, Z);
            }
            if (lane == 0) {
                const int items_b = seq_rows<GREEDY>(g, p.Gmax) * p.nseg;
                p.partial[((size_t)b * p.R + r) * p.S + sg] = out;
                __threadfence();
                unsigned old = atomicAdd(p.ticket + b, 1u);
                s_flag = (old == (unsigned)(items_b - 1));
            }
        }
        __syncthreads();
        const bool last = s_flag != 0;

        if (last) {
            // ---- this CTA saw the last segment of sequence b: merge partials, accept, scan ----
            __threadfence();
            const int rows_b = seq_rows<GREEDY>(g, p.Gmax);
            for (int l2 = warp; l2 < rows_b; l2 += kWarps) {
                const int r2 = (l2 <= g) ? l2 : p.Gmax + 1 + (l2 - g - 1);
                const float2* pp = p.partial + ((size_t)b * p.R + r2) * p.S;
                float2 st;
                if (GREEDY) {
                    ArgMax a{-INFINITY, INT_MAX};
                    for (int q = lane; q < p.nseg; q += 32) {
                        float2 v = __ldcg(pp + q);
                        a = better(a, ArgMax{v.x, __float_as_int(v.y)});
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        ArgMax t{__shfl_xor_sync(0xffffffffu, a.m, o), __shfl_xor_sync(0xffffffffu, a.idx, o)};
                        a = better(a, t);
                    }
                    if (a.idx == INT_MAX) a.idx = 0;          // row of -inf / NaN only
                    st = make_float2(a.m, __int_as_float(a.idx));
                } else {
                    Online o2{-INFINITY, 0.f};
                    for (int q = lane; q < p.nseg; q += 32) {
                        float2 v = __ldcg(pp + q);
                        o2.raise_to(v.x, p.c);
                        o2.s += v.y * rescale(v.x, o2.m, p.c);
                    }
                    float M = warp_max(o2.m);
                    float Z = warp_sum(o2.s * rescale(o2.m, M, p.c));
                    st = make_float2(M, Z);
                }
                if (lane == 0) {
                    s_stats[r2] = st;
                    p.row_stats[(size_t)b * p.R + r2] = st;
                }
            }
            __syncthreads();
            if (warp == 0) {
                const int j = lane;
                const bool valid = j < g;
                int st_bits = (p.gamma[b] < 0 || p.gamma[b] > p.Gmax) ? BS_DEV_BAD_GAMMA : 0;
                bool acc = false;
                float pj = 0.f, qj = 0.f;
                if (valid) {
                    const int x = p.tokens[(size_t)b * p.Gmax + j];
                    const bool bad = x < 0 || x >= p.V;
                    if (bad) st_bits |= BS_DEV_BAD_TOKEN;
                    const float2 ts = s_stats[j];
                    if (GREEDY) {
                        acc = !bad && x == __float_as_int(ts.y);
                    } else {
                        const float2 ds = s_stats[p.Gmax + 1 + j];
                        if (!(ts.y > 0.f) || !(ds.y > 0.f) || !isfinite(ts.y) || !isfinite(ds.y) ||
                            !isfinite(ts.x) || !isfinite(ds.x))
                            st_bits |= BS_DEV_NONFINITE;
                        if (!bad) {
                            const float tl = Elem<T>::load(row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, j, p.V) + x);
                            const float dl = Elem<T>::load(row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, j, p.V) + x);
                            // log2 of the two probabilities; the ratio is formed in the log domain
                            const float lp = (tl - ts.x) * p.c - log2f(ts.y);
                            const float lq = (dl - ds.x) * p.c - log2f(ds.y);
                            pj = exp2f(lp);
                            qj = exp2f(lq);
                            const float u = p.u_accept[(size_t)b * p.Gmax + j];
                            // r <= min{1, P/Q}; Q(x) = 0 counts as an infinite ratio
                            acc = (lq == -INFINITY) ? true : (u <= fminf(1.f, exp2f(lp - lq)));
                        }
                    }
                }
                if (!GREEDY && !valid && j == g) {   // the bonus row's normaliser is used by the resampler
                    const float2 ts = s_stats[g];
                    if (!(ts.y > 0.f) || !isfinite(ts.y) || !isfinite(ts.x)) st_bits |= BS_DEV_NONFINITE;
                }
                const unsigned accmask = __ballot_sync(0xffffffffu, valid && acc);
                const unsigned validmask = (g >= 32) ? 0xffffffffu : ((1u << g) - 1u);
                const unsigned rej = ~accmask & validmask;          // first zero among the valid bits
                const int tau = rej ? (__ffs(rej) - 1) : g;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) st_bits |= __shfl_xor_sync(0xffffffffu, st_bits, o);
                if (j < p.Gmax) {
                    if (p.p_tok) p.p_tok[(size_t)b * p.Gmax + j] = valid ? pj : 0.f;
                    if (p.q_tok) p.q_tok[(size_t)b * p.Gmax + j] = valid ? qj : 0.f;
                }
                if (lane == 0) {
                    p.accept_len[b] = tau;
                    p.status[b] = st_bits;
                    p.ticket[b] = 0u;                // leave the counter clear for the next call
                }
            }
        }
        __syncthreads();
    }
}

static int g_occ[4][64];     // resident CTAs per SM per kernel variant, per device (0 = not queried)
static int g_sms[64];

int sm_count() {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!g_sms[dev]) cudaDeviceGetAttribute(&g_sms[dev], cudaDevAttrMultiProcessorCount, dev);
    return g_sms[dev] > 0 ? g_sms[dev] : 148;
}

template <typename T, bool GREEDY>
static bs_status launch_verify(const VerifyParams& p, int variant, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    const size_t smem = sizeof(int) * (size_t)(p.B + 1);
    if (!g_occ[variant][dev]) {
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, verify_kernel<T, GREEDY>, kThreads,
                                                          sizeof(int) * (BS_MAX_BATCH + 1)) != cudaSuccess || occ < 1)
            occ = 1;
        g_occ[variant][dev] = occ;
    }
    const long long upper = (long long)p.B * (GREEDY ? p.Gmax + 1 : p.R) * p.nseg;
    long long grid = (long long)sm_count() * g_occ[variant][dev];
    if (grid > upper) grid = upper;
    if (grid < 1) grid = 1;
    verify_kernel<T, GREEDY><<<(unsigned)grid, kThreads, smem, st>>>(p);
    return cuda_status(cudaGetLastError());
}

}  // namespace bs

using namespace bs;

extern "C" const char* bs_status_string(bs_status s) {
    switch (s) {
        case BS_OK: return "ok";
        case BS_ERR_INVALID_ARG: return "invalid argument";
        case BS_ERR_CUDA: return "CUDA error";
        case BS_ERR_UNSUPPORTED: return "unsupported";
        case BS_ERR_WORKSPACE: return "workspace too small or misaligned";
        case BS_ERR_TIMEOUT: return "device-side wait timed out";
        case BS_ERR_DEVICE_DATA: return "device data error";
    }
    return "unknown";
}

static bool sizes_ok(int B, int Gmax, int V) {
    return B >= 1 && B <= BS_MAX_BATCH && Gmax >= 0 && Gmax <= BS_MAX_GAMMA && V >= 1 && V <= (1 << 20);
}

extern "C" size_t bs_workspace_bytes(int B, int Gmax, int V) {
    if (!sizes_ok(B, Gmax, V)) return 0;
    return workspace_layout(B, Gmax, V).total;
}

extern "C" bs_status bs_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || workspace_bytes == 0) return BS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return BS_ERR_WORKSPACE;
    return cuda_status(cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)));
}

extern "C" bs_status bs_get_device_status(const void* workspace, size_t workspace_bytes, int B, int Gmax, int V,
                                          int32_t* host_status, void* stream) {
    if (!workspace || !host_status || !sizes_ok(B, Gmax, V)) return BS_ERR_INVALID_ARG;
    const Workspace w = workspace_layout(B, Gmax, V);
    if (workspace_bytes < w.total) return BS_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(host_status, static_cast<const char*>(workspace) + w.off_status,
                                    sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return BS_ERR_CUDA;
    for (int b = 0; b < B; ++b)
        if (host_status[b]) return BS_ERR_DEVICE_DATA;
    return BS_OK;
}

extern "C" bs_status bs_softmax_verify(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                       const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                       float temperature, int B, int Gmax, int V,
                                       int32_t* accept_len, float* p_tok, float* q_tok,
                                       void* workspace, size_t workspace_bytes, void* stream) {
    if (!sizes_ok(B, Gmax, V)) return (B < 1 || Gmax < 0 || V < 1) ? BS_ERR_INVALID_ARG : BS_ERR_UNSUPPORTED;
    if (dtype != BS_F32 && dtype != BS_BF16) return BS_ERR_INVALID_ARG;
    if (!(temperature >= 0.f) || !isfinite(temperature)) return BS_ERR_INVALID_ARG;
    const bool greedy = temperature == 0.f;
    if (!target_logits || !gamma || !accept_len || !workspace) return BS_ERR_INVALID_ARG;
    if (Gmax > 0 && !draft_tokens) return BS_ERR_INVALID_ARG;
    if (!greedy && Gmax > 0 && (!draft_logits || !u_accept)) return BS_ERR_INVALID_ARG;
    const size_t es = dtype == BS_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(target_logits) % es) || (reinterpret_cast<uintptr_t>(draft_logits) % es))
        return BS_ERR_INVALID_ARG;
    const Workspace w = workspace_layout(B, Gmax, V);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) return BS_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    VerifyParams p;
    p.target = target_logits; p.draft = draft_logits; p.tokens = draft_tokens; p.gamma = gamma;
    p.u_accept = u_accept; p.accept_len = accept_len; p.p_tok = p_tok; p.q_tok = q_tok;
    p.ticket = reinterpret_cast<uint32_t*>(ws + w.off_ticket_verify);
    p.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    p.row_stats = reinterpret_cast<float2*>(ws + w.off_row_stats);
    p.partial = reinterpret_cast<float2*>(ws + w.off_partial);
    p.B = B; p.Gmax = Gmax; p.V = V; p.R = w.R; p.S = w.S;
    p.seg = seg_elems(dtype);
    p.nseg = div_up(V, p.seg);
    p.c = greedy ? 1.f : kLog2e / temperature;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == BS_F32)
        return greedy ? launch_verify<float, true>(p, 0, st) : launch_verify<float, false>(p, 1, st);
    return greedy ? launch_verify<__nv_bfloat16, true>(p, 2, st) : launch_verify<__nv_bfloat16, false>(p, 3, st);
}
