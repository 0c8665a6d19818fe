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
};
constexpr int kResidVerify = 0, kResidDraft = 1;

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

template <typename T>
bs_status launch_residual_stream(const ResidParams& p, cudaStream_t st);      // pipelined kernel, aligned rows

bs_status run_draft_resample(const void* draft_logits, bs_dtype dtype, int position, const int32_t* gamma,
                             const float* u_draft, float temperature, int B, int Gmax, int V, int32_t* draft_tokens,
                             void* workspace, size_t workspace_bytes, void* stream);

}  // namespace bs
