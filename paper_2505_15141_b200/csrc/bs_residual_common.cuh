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
};

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

}  // namespace bs
