// Pieces shared by the two row-statistics kernels (the pipelined one for 16-byte aligned rows and
// the generic one): the online-softmax state, partial merging, and the accept / first-rejection
// step of Algorithm 6 run by one warp per sequence.
#pragma once

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
    uint32_t* ticket;        // [B]
    uint32_t* ticket_row;    // [B, R]
    int32_t* status;         // [B]
    int32_t* abort_flag;     // [1]
    float2* row_stats;       // [B, R]
    float2* partial;         // [B, R, S]
    int B, Gmax, V, R, S;
    int nseg, seg;           // segments per row and elements per segment for this dtype
    float c;                 // log2(e) / temperature
    // Which rows a sequence contributes (pipelined kernel only):
    //   kModeVerify   target rows 0..g and draft rows 0..g-1 (target rows only in greedy mode)
    //   kModeDraft    the one draft row `position` (if position < g): its statistics go to the
    //                 draft slot of that position, no accept test; greedy: the arg-max is the token
    //   kModeDrafted  target rows 0..g only; the draft statistics are those kModeDraft left
    int mode, position;
    uint32_t* draft_ready;   // [B] bit j set: the statistics of draft row j are in row_stats
    int32_t* draft_out;      // kModeDraft, greedy: [B, Gmax] drafted tokens (entry [b, position] written)
};
constexpr int kModeVerify = 0, kModeDraft = 1, kModeDrafted = 2;

struct ArgMax {
    float m;
    int idx;
};
__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b) {      // larger value, then lower index
    return (b.m > a.m || (b.m == a.m && b.idx < a.idx)) ? b : a;
}
__device__ __forceinline__ ArgMax warp_best(ArgMax a) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ArgMax t{__shfl_xor_sync(0xffffffffu, a.m, o), __shfl_xor_sync(0xffffffffu, a.idx, o)};
        a = better(a, t);
    }
    return a;
}

// Running (m, s) of one thread: s = sum over seen x of exp2((x - m) * c).
struct Online {
    float m, s;
    __device__ __forceinline__ void raise_to(float mc, float c) {
        if (mc > m) { s *= rescale(m, mc, c); m = mc; }
    }
    __device__ __forceinline__ void merge(float m2, float s2, float c) {
        raise_to(m2, c);
        s += s2 * rescale(m2, m, c);
    }
};
__device__ __forceinline__ float2 warp_merge(Online o, float c) {    // fixed order; result in every lane
    const float M = warp_max(o.m);
    const float Z = warp_sum(o.s * rescale(o.m, M, c));
    return make_float2(M, Z);
}

template <typename T> __device__ __forceinline__ uint4 neg_inf_vec();
template <> __device__ __forceinline__ uint4 neg_inf_vec<float>() {
    return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
}
template <> __device__ __forceinline__ uint4 neg_inf_vec<__nv_bfloat16>() {
    return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
}

template <int N>
__device__ __forceinline__ float chunk_max_f32(const uint4 (&v)[N]) {
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < N; ++k)
        m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(v[k].x), __uint_as_float(v[k].y)),
                           fmaxf(__uint_as_float(v[k].z), __uint_as_float(v[k].w))));
    return m;
}
template <int N>
__device__ __forceinline__ float chunk_max_bf16(const uint4 (&v)[N]) {
    // packed max on the raw bf16 pairs: two elements per instruction
    __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&v[0].x);
#pragma unroll
    for (int k = 0; k < N; ++k) {
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].x));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].y));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].z));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&v[k].w));
    }
    const uint32_t w = *reinterpret_cast<uint32_t*>(&m2);
    return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
template <typename T, int N> struct ChunkMax;
template <int N> struct ChunkMax<float, N> {
    __device__ static __forceinline__ float of(const uint4 (&v)[N]) { return chunk_max_f32<N>(v); }
};
template <int N> struct ChunkMax<__nv_bfloat16, N> {
    __device__ static __forceinline__ float of(const uint4 (&v)[N]) { return chunk_max_bf16<N>(v); }
};

// Adds N 128-bit vectors of logits to the running state with one exp per element: the chunk
// maximum is found first, the running sum rescaled once if it rises.  Slots filled with -inf
// contribute nothing.
template <typename T, int N>
__device__ __forceinline__ void online_add(Online& on, const uint4 (&v)[N], float c) {
    constexpr int kVec = Elem<T>::kVec;
    on.raise_to(ChunkMax<T, N>::of(v), c);
    if (on.m > -INFINITY) {
        const float nm = -on.m * c;
        float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
        for (int k = 0; k < N; ++k) {
            float f[kVec];
            Elem<T>::unpack(v[k], f);
#pragma unroll
            for (int q = 0; q < kVec; q += 2) {
                acc0 += ex2(fmaf(f[q], c, nm));
                acc1 += ex2(fmaf(f[q + 1], c, nm));
            }
        }
        // nm is the rounded product: the terms above are 2^((x - m) c) times 2^dl with dl = m c + nm, the
        // rounding error of the product, which one FMA gives exactly.  Undone to first order (dl^2 < 1e-9),
        // so that the sum does not carry an error that grows with |m| / temperature.
        const float dl = fmaf(on.m, c, nm);
        on.s = fmaf(acc0 + acc1, fmaf(-dl, 0.69314718f, 1.f), on.s);
    }
}

template <typename T, int N>
__device__ __forceinline__ void argmax_add(ArgMax& am, const uint4 (&v)[N], int first_elem, int vec_stride) {
    constexpr int kVec = Elem<T>::kVec;
#pragma unroll
    for (int k = 0; k < N; ++k) {
        float f[kVec];
        Elem<T>::unpack(v[k], f);
        const int ei = first_elem + k * vec_stride;
#pragma unroll
        for (int q = 0; q < kVec; ++q)
            if (f[q] > am.m) { am.m = f[q]; am.idx = ei + q; }
    }
}

// Items of sequence b: rows * segments.  An out-of-range gamma is processed as gamma = 0.
__device__ __forceinline__ int clamp_gamma(int g, int Gmax) { return (g < 0 || g > Gmax) ? 0 : g; }
template <bool GREEDY>
__device__ __forceinline__ int seq_rows(int g, int Gmax) {
    g = clamp_gamma(g, Gmax);
    return GREEDY ? g + 1 : 2 * g + 1;
}
// local row index (0..rows_b-1) -> row slot in [0, R): target rows first, then draft rows
__device__ __forceinline__ int row_slot(int lr, int g, int Gmax) { return lr <= g ? lr : Gmax + 1 + (lr - g - 1); }

// The same three questions for any mode of the pipelined kernel (g already clamped).
template <bool GREEDY>
__device__ __forceinline__ int mode_rows(const VerifyParams& p, int g) {
    if (p.mode == kModeDraft) return p.position < g ? 1 : 0;
    if (p.mode == kModeDrafted) return g + 1;
    return GREEDY ? g + 1 : 2 * g + 1;
}
__device__ __forceinline__ int mode_slot(const VerifyParams& p, int lr, int g) {
    if (p.mode == kModeDraft) return p.Gmax + 1 + p.position;
    return row_slot(lr, g, p.Gmax);                      // kModeDrafted: lr <= g, so the slot is lr
}
template <typename T>
__device__ __forceinline__ const T* mode_row(const VerifyParams& p, int b, int lr, int g) {
    if (p.mode == kModeDraft) return row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, p.position, p.V);
    return lr <= g ? row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, lr, p.V)
                   : row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, lr - g - 1, p.V);
}

// One warp merges the nseg partial slots of a row (all lanes return the result).
template <bool GREEDY>
__device__ __forceinline__ float2 merge_row_partials(const float2* pp, int nseg, float c) {
    const int lane = threadIdx.x & 31;
    if (GREEDY) {
        ArgMax a{-INFINITY, INT_MAX};
        for (int q = lane; q < nseg; q += 32) {
            const float2 v = __ldcg(pp + q);
            a = better(a, ArgMax{v.x, __float_as_int(v.y)});
        }
        a = warp_best(a);
        if (a.idx == INT_MAX) a.idx = 0;                      // row of -inf / NaN only
        return make_float2(a.m, __int_as_float(a.idx));
    }
    Online o{-INFINITY, 0.f};
    for (int q = lane; q < nseg; q += 32) {
        const float2 v = __ldcg(pp + q);
        o.merge(v.x, v.y, c);
    }
    return warp_merge(o, c);
}

// Accept test and first-rejection scan for sequence b by one full warp (lane j = drafted position j),
// in two steps so that a caller can start the loads before it knows whether it will need them.
//
// accept_prefetch: everything that does not depend on the row statistics -- the drafted token, the
// two logits at that token, the uniform.
struct AcceptLoads {
    int x;              // drafted token of this lane's position (undefined if the position is not valid)
    float tl, dl, u;    // target / draft logit at x, uniform
    int bits;           // BS_DEV_BAD_TOKEN if x is out of range
};
template <typename T, bool GREEDY>
__device__ __forceinline__ AcceptLoads accept_prefetch(const VerifyParams& p, int b, int g) {
    const int j = threadIdx.x & 31;
    AcceptLoads a{0, 0.f, 0.f, 2.f, 0};
    if (j < g) {
        a.x = p.tokens[(size_t)b * p.Gmax + j];
        const bool bad = a.x < 0 || a.x >= p.V;
        if (bad) a.bits = BS_DEV_BAD_TOKEN;
        if (!GREEDY && !bad) {
            a.tl = Elem<T>::load(row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, j, p.V) + a.x);
            a.dl = Elem<T>::load(row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, j, p.V) + a.x);
            a.u = p.u_accept[(size_t)b * p.Gmax + j];
        }
    }
    return a;
}

// accept_finish: stats(r) returns the (max, Z) / (max, arg-max) pair of row slot r.  Writes
// accept_len, p_tok, q_tok and the status word.  graw = gamma[b] as read, g = clamp_gamma(graw).
template <typename T, bool GREEDY, typename StatsFn>
__device__ __forceinline__ void accept_finish(const VerifyParams& p, int b, int graw, int g, const AcceptLoads& a,
                                              StatsFn stats, int extra_bits = 0) {
    const int lane = threadIdx.x & 31;
    const int j = lane;
    const bool valid = j < g;
    int st_bits = ((graw != g) ? BS_DEV_BAD_GAMMA : 0) | a.bits | extra_bits;
    bool acc = false;
    float pj = 0.f, qj = 0.f;
    if (valid) {
        const bool bad = a.bits != 0;
        const float2 ts = stats(j);
        if (GREEDY) {
            acc = !bad && a.x == __float_as_int(ts.y);
        } else {
            const float2 ds = stats(p.Gmax + 1 + j);
            if (!(ts.y > 0.f) || !(ds.y > 0.f) || !isfinite(ts.y) || !isfinite(ds.y) || !isfinite(ts.x) ||
                !isfinite(ds.x))
                st_bits |= BS_DEV_NONFINITE;
            if (!bad) {
                // log2 of the two probabilities; the ratio is formed in the log domain
                const float lp = (a.tl - ts.x) * p.c - log2f(ts.y);
                const float lq = (a.dl - ds.x) * p.c - log2f(ds.y);
                pj = exp2f(lp);
                qj = exp2f(lq);
                // r <= min{1, P/Q}; Q(x) = 0 counts as an infinite ratio
                acc = (lq == -INFINITY) ? true : (a.u <= fminf(1.f, exp2f(lp - lq)));
            }
        }
        if (extra_bits & BS_DEV_DRAFT_MISSING) acc = false;   // no draft statistics: nothing is accepted
    }
    if (!GREEDY && j == g) {              // the bonus row's normaliser is used by the resampler
        const float2 ts = stats(g);
        if (!(ts.y > 0.f) || !isfinite(ts.y) || !isfinite(ts.x)) st_bits |= BS_DEV_NONFINITE;
    }
    const unsigned accmask = __ballot_sync(0xffffffffu, valid && acc);
    const unsigned validmask = (g >= 32) ? 0xffffffffu : ((1u << g) - 1u);
    const unsigned rej = ~accmask & validmask;               // first zero among the valid bits
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
    }
}

template <typename T, bool GREEDY, typename StatsFn>
__device__ __forceinline__ void accept_scan_warp(const VerifyParams& p, int b, StatsFn stats) {
    const int graw = p.gamma[b];
    const int g = clamp_gamma(graw, p.Gmax);
    const AcceptLoads a = accept_prefetch<T, GREEDY>(p, b, g);
    accept_finish<T, GREEDY>(p, b, graw, g, a, stats);
}

template <typename T, bool GREEDY>
bs_status launch_verify_stream(const VerifyParams& p, cudaStream_t st);   // pipelined kernel, aligned rows

bs_status run_verify(const void* target_logits, const void* draft_logits, bs_dtype dtype, const int32_t* draft_tokens,
                     const int32_t* gamma, const float* u_accept, float temperature, int B, int Gmax, int V,
                     int32_t* accept_len, float* p_tok, float* q_tok, void* workspace, size_t workspace_bytes,
                     void* stream, int mode, int position, int32_t* draft_out);

}  // namespace bs
