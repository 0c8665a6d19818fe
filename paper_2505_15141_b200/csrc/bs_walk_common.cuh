// Pieces shared by the two early-exit kernels (bs_verify_walk): the one whose CTA groups are thread-block
// clusters and talk through distributed shared memory, and the one whose groups talk through the workspace.
#pragma once

#include "bs_verify_common.cuh"
#include "bs_residual_level2.cuh"
#include "bs_pipeline.cuh"

namespace bs {

constexpr int kWkWarps = 16;
constexpr int kWkConsumers = kWkWarps * 32;
constexpr int kWkThreads = kWkConsumers + 64;                    // + producer warp + finisher warp
constexpr int kWkStages = 3;
constexpr int kWkRing = 8;                                       // events the consumers may run ahead of the finisher
constexpr int kWkVecPerThread = kSegBytes / 16 / kWkConsumers;   // 4
static_assert(kSegBytes == 2 * kResSegBytes && kWkWarps == kRsWarps, "one stage holds a segment or a pair of half segments");

constexpr int kItemStats = 0, kItemMass = 1, kItemEnd = 2, kItemAck = 3;

struct WalkParams {
    VerifyParams v;        // logits, tokens, uniforms, outputs of the accept test, statistics and partials
    ResidParams r;         // the same logits for the residual pass, its outputs, piece masses
    uint32_t* dec;         // [B] decision word: (positions decided << 1) | last one accepted
    int nG;                // CTAs per sequence
    int drafted;           // 1: the draft rows' statistics were left by bs_draft_sample: stream target rows only
    int look;              // cluster kernel: positions a sequence may be streamed past its last decided one
};

// Per-stage record, written by the producer.
struct WkMeta {
    int type, b, k;
    int row;               // stats: 0 = target row k, 1 = draft row k;  mass: 1 = target row only (bonus)
    int sg, nvec, flags;   // flags bit 0: first stage of a row piece, bit 1: last stage of a piece / of the CTA's share
    float kt, kd, at, ad;
};

// The cluster kernel: groups of nG = 2, 4 or 8 CTAs.  BS_ERR_UNSUPPORTED if this shape cannot be launched that
// way (the caller then uses the kernel that goes through the workspace).
template <typename T, bool GREEDY>
bs_status launch_walk_cluster(WalkParams& p, cudaStream_t st);

}  // namespace bs
