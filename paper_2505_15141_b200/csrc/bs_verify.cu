// bs_softmax_verify: entry point, plus the generic row-statistics kernel used when rows do not
// start on 16-byte boundaries (V * sizeof(element) not a multiple of 16).  Rows that do are
// handled by the pipelined kernel in bs_verify_stream.cu.  Algorithm 6 of the paper, second
// line and for-loop; softmax with temperature as in Section 2.
//
// Generic kernel: a work item is one segment of one valid row.  Every CTA builds the prefix sum
// of items per sequence in shared memory and the persistent grid strides over the flat item
// list.  Each item is read with a scalar head up to the next 16-byte boundary, a 128-bit body
// and a scalar tail, reduced to (max, sum exp) with one exp per logit, and written as a
// partial.  An arrival counter per sequence elects the CTA that merges the partials and runs
// the accept scan.
#include <atomic>
#include "bs_verify_common.cuh"

namespace bs {

constexpr int kUnroll = 4;      // 128-bit loads in flight per thread: one segment per trip

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
    pdl_enter();

    // ---- prefix sum of work items over the batch (every CTA, redundantly) ----
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
        const int g = clamp_gamma(p.gamma[b], p.Gmax);
        const bool is_target = lr <= g;
        const int r = row_slot(lr, g, p.Gmax);
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
            if (GREEDY) argmax_add<T, kUnroll>(am, v, e0 + head + (base + tid) * kVec, kThreads * kVec);
            else online_add<T, kUnroll>(on, v, p.c);
        }
        if (tid < n - tail0) {
            float x = Elem<T>::load(sp + tail0 + tid);
            if (GREEDY) { if (x > am.m) { am.m = x; am.idx = e0 + tail0 + tid; } }
            else if (x != -INFINITY) { on.raise_to(x, p.c); on.s += ex2((x - on.m) * p.c); }
        }

        // ---- block reduction (fixed order, deterministic) ----
        if (GREEDY) {
            am = warp_best(am);
            if (lane == 0) { s_m[warp] = am.m; s_i[warp] = am.idx; }
        } else {
            const float2 w = warp_merge(on, p.c);
            if (lane == 0) { s_m[warp] = w.x; s_s[warp] = w.y; }
        }
        __syncthreads();
        if (warp == 0) {
            float2 out;
            if (GREEDY) {
                ArgMax a{lane < kWarps ? s_m[lane] : -INFINITY, lane < kWarps ? s_i[lane] : INT_MAX};
                a = warp_best(a);
                out = make_float2(a.m, __int_as_float(a.idx));
            } else {
                Online o{lane < kWarps ? s_m[lane] : -INFINITY, lane < kWarps ? s_s[lane] : 0.f};
                out = warp_merge(o, p.c);
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
                const int r2 = row_slot(l2, g, p.Gmax);
                const float2 st = merge_row_partials<GREEDY>(p.partial + ((size_t)b * p.R + r2) * p.S, p.nseg, p.c);
                if (lane == 0) {
                    s_stats[r2] = st;
                    p.row_stats[(size_t)b * p.R + r2] = st;
                }
            }
            __syncthreads();
            if (warp == 0) {
                accept_scan_warp<T, GREEDY>(p, b, [&](int rr) { return s_stats[rr]; });
                if (lane == 0) p.ticket[b] = 0u;         // leave the counter clear for the next call
            }
        }
        __syncthreads();
    }
}

thread_local int g_last_cuda_error = 0;

static std::atomic<int> g_occ[4][64];     // resident CTAs per SM per kernel variant, per device (0 = not queried)
static std::atomic<int> g_sms[64];

int sm_count() {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    int n = g_sms[dev];
    if (!n) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        g_sms[dev] = n;
    }
    return n;
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
    return cuda_status(launch_pdl(verify_kernel<T, GREEDY>, (unsigned)grid, kThreads, smem, st, p));
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

extern "C" const char* bs_last_cuda_error(void) {
    return g_last_cuda_error ? cudaGetErrorString(static_cast<cudaError_t>(g_last_cuda_error)) : "no error";
}

static bool sizes_ok(int B, int Gmax, int V) {
    return B >= 1 && B <= BS_MAX_BATCH && Gmax >= 0 && Gmax <= BS_MAX_GAMMA && V >= 1 && V <= BS_MAX_VOCAB;
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
    int32_t aborted = 0;
    cudaError_t e = cudaMemcpyAsync(host_status, static_cast<const char*>(workspace) + w.off_status,
                                    sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(&aborted, static_cast<const char*>(workspace) + w.off_abort, sizeof(int32_t),
                            cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return BS_ERR_CUDA;
    if (aborted) return BS_ERR_TIMEOUT;
    for (int b = 0; b < B; ++b)
        if (host_status[b]) return BS_ERR_DEVICE_DATA;
    return BS_OK;
}

// Host side shared by bs_softmax_verify (kModeVerify), bs_softmax_verify_drafted (kModeDrafted) and
// the statistics pass of bs_draft_sample (kModeDraft: target_logits and accept_len unused,
// draft_out = the token array for greedy drafting).
bs_status bs::run_verify(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                         const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                         float temperature, int B, int Gmax, int V, int32_t* accept_len, float* p_tok, float* q_tok,
                         void* workspace, size_t workspace_bytes, void* stream, int mode, int position,
                         int32_t* draft_out) {
    if (!sizes_ok(B, Gmax, V)) return (B < 1 || Gmax < 0 || V < 1) ? BS_ERR_INVALID_ARG : BS_ERR_UNSUPPORTED;
    if (dtype != BS_F32 && dtype != BS_BF16) return BS_ERR_INVALID_ARG;
    if (!(temperature >= 0.f) || !isfinite(temperature)) return BS_ERR_INVALID_ARG;
    const bool greedy = temperature == 0.f;
    if (!gamma || !workspace) return BS_ERR_INVALID_ARG;
    if (mode == kModeDraft) {
        if (!draft_logits || position < 0 || position >= Gmax || (greedy && !draft_out)) return BS_ERR_INVALID_ARG;
    } else {
        if (!target_logits || !accept_len) return BS_ERR_INVALID_ARG;
        if (Gmax > 0 && !draft_tokens) return BS_ERR_INVALID_ARG;
        if (!greedy && Gmax > 0 && (!draft_logits || !u_accept)) return BS_ERR_INVALID_ARG;
    }
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
    p.ticket_row = reinterpret_cast<uint32_t*>(ws + w.off_ticket_row);
    p.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    p.abort_flag = reinterpret_cast<int32_t*>(ws + w.off_abort);
    p.row_stats = reinterpret_cast<float2*>(ws + w.off_row_stats);
    p.partial = reinterpret_cast<float2*>(ws + w.off_partial);
    p.B = B; p.Gmax = Gmax; p.V = V; p.R = w.R; p.S = w.S;
    p.seg = seg_elems(dtype);
    p.nseg = div_up(V, p.seg);
    p.c = greedy ? 1.f : kLog2e / temperature;
    p.mode = mode; p.position = position; p.draft_out = draft_out;
    p.draft_ready = p.ticket_row;          // the per-row counters' slot: the pipelined kernel counts per sequence
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // rows start on 16-byte boundaries: bulk-copy pipeline; otherwise the generic kernel
    const bool aligned = ((size_t)V * es) % 16 == 0 && (reinterpret_cast<uintptr_t>(target_logits) & 15) == 0 &&
                         (reinterpret_cast<uintptr_t>(draft_logits) & 15) == 0;
    if (!aligned && mode != kModeVerify) return BS_ERR_UNSUPPORTED;   // the drafting path needs aligned rows
    if (aligned) {
        if (dtype == BS_F32)
            return greedy ? launch_verify_stream<float, true>(p, st) : launch_verify_stream<float, false>(p, st);
        return greedy ? launch_verify_stream<__nv_bfloat16, true>(p, st)
                      : launch_verify_stream<__nv_bfloat16, false>(p, st);
    }
    if (dtype == BS_F32)
        return greedy ? launch_verify<float, true>(p, 0, st) : launch_verify<float, false>(p, 1, st);
    return greedy ? launch_verify<__nv_bfloat16, true>(p, 2, st) : launch_verify<__nv_bfloat16, false>(p, 3, st);
}

extern "C" bs_status bs_softmax_verify(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                       const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                       float temperature, int B, int Gmax, int V,
                                       int32_t* accept_len, float* p_tok, float* q_tok,
                                       void* workspace, size_t workspace_bytes, void* stream) {
    return run_verify(target_logits, draft_logits, dtype, draft_tokens, gamma, u_accept, temperature, B, Gmax, V,
                      accept_len, p_tok, q_tok, workspace, workspace_bytes, stream, kModeVerify, 0, nullptr);
}
