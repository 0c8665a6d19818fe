// bs_draft_sample and bs_softmax_verify_drafted: the drafting step of Algorithm 6 (first line,
// x~_{j+1} ~ Q(. | pt, x~_{1:j})) on the device, and the verification that re-uses what drafting
// already computed.
//
// A draft model produces its rows one position at a time, and each row has to be normalised to
// draw its token.  bs_draft_sample does that with the library's two streaming kernels: the
// statistics kernel in its drafting mode reads the row once and leaves (max, Z) in the draft slot of
// that position; the resampling kernel in its drafting mode turns the row into one token by inverse
// CDF.  bs_softmax_verify_drafted then streams the target rows only: of each draft row it needs
// the statistics, which are there, and the one logit of the drafted token.
#include "bs_verify_common.cuh"
#include "bs_residual_common.cuh"

using namespace bs;

extern "C" bs_status bs_draft_sample(const void* draft_logits, bs_dtype dtype, int position, const int32_t* gamma,
                                     const float* u_draft, float temperature, int B, int Gmax, int V,
                                     int32_t* draft_tokens, void* workspace, size_t workspace_bytes, void* stream) {
    if (!draft_tokens) return BS_ERR_INVALID_ARG;
    if (!(temperature >= 0.f) || !isfinite(temperature)) return BS_ERR_INVALID_ARG;
    const bool greedy = temperature == 0.f;
    if (!greedy && !u_draft) return BS_ERR_INVALID_ARG;
    const bs_status s = run_verify(nullptr, draft_logits, dtype, nullptr, gamma, nullptr, temperature, B, Gmax, V,
                                   nullptr, nullptr, nullptr, workspace, workspace_bytes, stream, kModeDraft, position,
                                   draft_tokens);
    if (s != BS_OK || greedy) return s;          // greedy: the arg-max found by the statistics pass is the token
    return run_draft_resample(draft_logits, dtype, position, gamma, u_draft, temperature, B, Gmax, V, draft_tokens,
                              workspace, workspace_bytes, stream);
}

extern "C" bs_status bs_softmax_verify_drafted(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                               const int32_t* draft_tokens, const int32_t* gamma,
                                               const float* u_accept, float temperature, int B, int Gmax, int V,
                                               int32_t* accept_len, float* p_tok, float* q_tok, void* workspace,
                                               size_t workspace_bytes, void* stream) {
    return run_verify(target_logits, draft_logits, dtype, draft_tokens, gamma, u_accept, temperature, B, Gmax, V,
                      accept_len, p_tok, q_tok, workspace, workspace_bytes, stream, kModeDrafted, 0, nullptr);
}
