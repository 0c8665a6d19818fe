// Pieces shared by the two resampling kernels (the pipelined one for 16-byte aligned rows and the
// generic one): parameters and the residual mass of Algorithm 6's else-branch,
// r_v = max(0, P(v) - Q(v)), or P(v) alone for the bonus token.
#pragma once

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
    int32_t* abort_flag;
    const float2* row_stats;
    float* resid_partial;
    int B, Gmax, V, R, S;
    int nseg, seg;
    float c;
    // kResidVerify: Algorithm 6's resampling / bonus step.  kResidDraft: the drafting step -- for
    // every sequence with position < gamma_b one token from softmax(draft row `position`), uniform
    // u_resample[b, position] (a [B, Gmax] array in this mode), written to draft_out[b, position];
    // the row's statistics are read from its draft slot.
    int mode, position;
    int32_t* draft_out;
    uint32_t* draft_ready;   // kResidDraft: [B] word of the drafted positions; bit 31 reports a row that could not be sampled
};
constexpr int kResidVerify = 0, kResidDraft = 1;

// Norm([P - Q]_+) needs a positive total.  The total is the probability of reaching this step at all
// (1 - sum_v min(P, Q)), and below about 1e-6 what fp32 holds of P - Q is rounding noise of the two
// normalisers, not a direction: a total at or below this floor counts as "no mass" and the token is
// drawn from the target row instead (status bit BS_DEV_RESIDUAL_FALLBACK).
constexpr double kResidualFloor = 1.0 / 262144.0;            // 2^-18

// Mass of one element.  kt / kd fold the row max and normaliser into the exponent, p = at * 2^(x*c + kt):
// kt is the rounded -(m c + log2 Z); at = 2^(what the two roundings lost) to first order, so that P and Q
// are not scaled apart by an error that grows with |m| / temperature.
struct MassFn {
    float c, kt, kd;
    float at, ad;
    bool bonus;
    __device__ __forceinline__ float operator()(float xt, float xd) const {
        const float pv = at * ex2(fmaf(xt, c, kt));
        if (bonus) return pv;
        const float qv = ex2(fmaf(xd, c, kd));
        return fmaxf(0.f, fmaf(-ad, qv, pv));
    }
    // row statistics (raw max m, sum Z relative to m) -> (k, a)
    __device__ static __forceinline__ void fold(float m, float Z, float c, float& k, float& a) {
        const float p1 = m * c;
        const float d1 = fmaf(m, c, -p1);                     // m c = p1 + d1 exactly
        const float l = log2f(Z);
        const float sum = p1 + l;
        const float bb = sum - p1;
        const float d2 = (p1 - (sum - bb)) + (l - bb);        // p1 + l = sum + d2 exactly
        k = -sum;
        a = fmaf(-(d1 + d2), 0.69314718f, 1.f);               // 2^-(d1 + d2), |d1 + d2| < 1e-4
        if (!(fabsf(d1 + d2) < 1.f)) a = 1.f;                 // non-finite statistics: reported elsewhere
    }
};

template <typename T>
bs_status launch_residual_stream(const ResidParams& p, cudaStream_t st);      // pipelined kernel, aligned rows

bs_status run_draft_resample(const void* draft_logits, bs_dtype dtype, int position, const int32_t* gamma,
                             const float* u_draft, float temperature, int B, int Gmax, int V, int32_t* draft_tokens,
                             void* workspace, size_t workspace_bytes, void* stream);

}  // namespace bs
