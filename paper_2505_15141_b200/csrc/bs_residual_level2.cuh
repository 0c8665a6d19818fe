// Pieces of the pipelined resampling kernel that other kernels share: the geometry of a segment
// (16 consumer warps, one 1 KB piece of each row per warp), the per-sequence facts, the masses of
// a 16-byte vector, and level 2 -- the inverse CDF over the piece masses by one warp.
#pragma once

#include "bs_residual_common.cuh"

#include <limits.h>

namespace bs {

constexpr int kRsWarps = kResSubSegs;                          // 16 consumer warps, one piece each
constexpr int kRsConsumers = kRsWarps * 32;
constexpr int kRsThreads = kRsConsumers + 64;                  // + producer warp + finisher warp
constexpr int kRsStageBytes = 2 * kResSegBytes;                // target half, draft half
constexpr int kRsMaxStages = 3;
constexpr int kRsPieceBytes = kResSegBytes / kRsWarps;         // 1 KB of each row per warp and item
constexpr int kRsPieceVecs = kRsPieceBytes / 16;               // 64
constexpr int kRsVecPerLane = kRsPieceVecs / 32;               // 2
static_assert(kRsVecPerLane * 32 * 16 * kRsWarps == kResSegBytes, "pieces must tile the segment");

struct RsMeta {
    int b, sg;
    int nvec;        // valid 16-byte vectors in the first half of the slot
    int nvec2;       // ... in the second half: the draft row's segment, or segment sg + 1 of a row sampled alone
    int flags;       // bit 0: bonus (target row only), bit 1: last item of this sequence in the CTA's range
    float kt, kd;    // p_v = at 2^(x_t c + kt), q_v = ad 2^(x_d c + kd)
    float at, ad;
};

// Per-sequence facts every role derives the same way.
struct RsSeq {
    int tau, bonus, wgt;     // weight of one item: 2 (row pair) or 1 (target row only)
};
__device__ __forceinline__ RsSeq rs_seq(const ResidParams& p, int b) {
    int g = p.gamma[b];
    if (g < 0 || g > p.Gmax) g = 0;
    RsSeq s;
    if (p.mode == kResidDraft) {          // drafting: sample from the draft row `position` alone, if the sequence drafts it
        s.tau = p.position;
        s.bonus = 1;
        s.wgt = p.position < g ? 1 : 0;
        return s;
    }
    s.tau = max(0, min(p.accept_len[b], g));
    s.bonus = s.tau >= g;
    s.wgt = s.bonus ? 1 : 2;
    return s;
}
// Items of a sequence in the pipelined kernel.  A slot has two 16 KB halves: for a row pair they hold
// the same segment of the target and of the draft row, for a row sampled alone two consecutive
// segments of it, so that every item keeps up to 32 KB in flight (with one segment per item the
// CTAs whose sequences were all accepted moved half the bytes per item and finished last).
__device__ __forceinline__ int rs_nitems(const RsSeq& s, int nseg) {
    return s.wgt <= 0 ? 0 : (s.bonus ? (nseg + 1) >> 1 : nseg);
}
__device__ __forceinline__ int rs_first_seg(const RsSeq& s, int item) { return s.bonus ? 2 * item : item; }
// Items [i0, i1) of a sequence with `nitems` items that lie in the CTA's range [lo, hi); pre = index of its first item.
__device__ __forceinline__ void rs_items(int pre, int nitems, int lo, int hi, int& i0, int& i1) {
    i0 = max(lo, pre) - pre;
    i1 = min(hi, pre + nitems) - pre;
    if (i1 < i0) i1 = i0;
}

// The row that is sampled alone (or minus the draft row) and the slot of its statistics.
template <typename T>
__device__ __forceinline__ const T* rs_trow(const ResidParams& p, int b, const RsSeq& sq) {
    return p.mode == kResidDraft ? row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, p.position, p.V)
                                 : row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, sq.tau, p.V);
}
__device__ __forceinline__ int rs_tslot(const ResidParams& p, const RsSeq& sq) {
    return p.mode == kResidDraft ? p.Gmax + 1 + p.position : sq.tau;
}

template <typename T>
struct RsElems {
    static constexpr int kVec = Elem<T>::kVec;
    // masses of one 16-byte vector of the row pair
    __device__ static __forceinline__ void masses(const uint4& a, const uint4& d, const MassFn& f, float (&r)[kVec]) {
        float ft[kVec], fd[kVec];
        Elem<T>::unpack(a, ft);
        Elem<T>::unpack(d, fd);
#pragma unroll
        for (int q = 0; q < kVec; ++q) r[q] = f(ft[q], fd[q]);
    }
};

__device__ __forceinline__ double warp_scan_incl(double v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Level 2 for sequence b by one warp.  `f` has the sequence's constants.
template <typename T>
__device__ void rs_level2(const ResidParams& p, int b, const RsSeq sq, MassFn f) {
    constexpr int kVec = Elem<T>::kVec;
    const int lane = threadIdx.x & 31;
    const T* tp = rs_trow<T>(p, b, sq);
    const T* dp = f.bonus ? tp : row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, sq.tau, p.V);
    const float* pm = p.resid_partial + (size_t)b * p.S;
    const int nsub = p.nseg * kRsWarps;
    const int per = div_up(nsub, 32);
    const int s0 = min(nsub, lane * per), s1 = min(nsub, s0 + per);
    int bits = 0;

    // ---- piece masses: fp64 sum per lane in index order, then a scan over the lanes ----
    double mine = 0.0;
    int lastpos = -1;
    for (int i = s0; i < s1; ++i) {
        const float m = __ldcg(pm + i);
        mine += (double)m;
        if (m > 0.f) lastpos = i;
    }
    double incl = warp_scan_incl(mine);
    double Rtot = __shfl_sync(0xffffffffu, incl, 31);
    const float u = p.mode == kResidDraft ? p.u_resample[(size_t)b * p.Gmax + p.position] : p.u_resample[b];
    int tok = -1;

    if (Rtot > (f.bonus ? 0.0 : kResidualFloor) && isfinite(Rtot)) {
        const double target = (double)u * Rtot;
        double excl = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) excl = 0.0;
        int ps = -1;
        double before = 0.0;
        // the lane in whose pieces the crossing falls; its pieces are then searched by the whole
        // warp, 32 at a time (one load latency per round instead of one per piece)
        const unsigned cross = __ballot_sync(0xffffffffu, incl > target && !(excl > target));
        if (cross) {
            const int L = __ffs(cross) - 1;
            const int c0 = __shfl_sync(0xffffffffu, s0, L), c1 = __shfl_sync(0xffffffffu, s1, L);
            double run0 = __shfl_sync(0xffffffffu, excl, L);  // mass in front of the lane's pieces
            int lastp = -1;                                   // so far: the last piece with mass
            double lastbefore = 0.0;
            for (int r0 = c0; r0 < c1 && ps < 0; r0 += 32) {
                const int i = r0 + lane;
                const double m = i < c1 ? (double)__ldcg(pm + i) : 0.0;
                const double sc = warp_scan_incl(m);
                double sx = __shfl_up_sync(0xffffffffu, sc, 1);
                if (lane == 0) sx = 0.0;
                // the first piece whose end passes the target
                const unsigned hit = __ballot_sync(0xffffffffu, run0 + sc > target && !(run0 + sx > target) && m > 0.0);
                if (hit) {
                    const int src = __ffs(hit) - 1;
                    ps = __shfl_sync(0xffffffffu, i, src);
                    before = __shfl_sync(0xffffffffu, run0 + sx, src);
                } else {
                    const unsigned pos = __ballot_sync(0xffffffffu, m > 0.0);
                    if (pos) {
                        const int src = 31 - __clz(pos);
                        lastp = __shfl_sync(0xffffffffu, i, src);
                        lastbefore = __shfl_sync(0xffffffffu, run0 + sx, src);
                    }
                    run0 += __shfl_sync(0xffffffffu, sc, 31);
                }
            }
            if (ps < 0 && lastp >= 0) { ps = lastp; before = lastbefore; }   // rounding only
        }
        // the lane that found the piece tells the others
        const unsigned found = __ballot_sync(0xffffffffu, ps >= 0);
        bool take_last = false;
        if (found) {
            const int src = __ffs(found) - 1;
            ps = __shfl_sync(0xffffffffu, ps, src);
            before = __shfl_sync(0xffffffffu, before, src);
        } else {                                              // rounding only: the last piece with mass, its last token
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lastpos = max(lastpos, __shfl_xor_sync(0xffffffffu, lastpos, o));
            ps = lastpos;
            take_last = true;
        }
        if (ps >= 0) {
            const double t_in = target - before;
            const int sg = ps / kRsWarps, w = ps - sg * kRsWarps;
            const int e0 = sg * p.seg;
            const int nvec = min(p.seg, p.V - e0) / kVec;
            double pbase = 0.0;
            int lastel = -1;
#pragma unroll
            for (int q = 0; q < kRsVecPerLane; ++q) {
                const int iv = w * kRsPieceVecs + q * 32 + lane;
                float r[kVec];
#pragma unroll
                for (int k = 0; k < kVec; ++k) r[k] = 0.f;
                if (iv < nvec) {
                    const uint4 a = __ldcg(reinterpret_cast<const uint4*>(tp + e0) + iv);
                    const uint4 d = f.bonus ? a : __ldcg(reinterpret_cast<const uint4*>(dp + e0) + iv);
                    RsElems<T>::masses(a, d, f, r);
                }
                float vs = 0.f;
#pragma unroll
                for (int k = 0; k < kVec; ++k) {
                    vs += r[k];
                    if (r[k] > 0.f) lastel = e0 + iv * kVec + k;
                }
                const double sc = warp_scan_incl((double)vs);
                double sx = __shfl_up_sync(0xffffffffu, sc, 1);
                if (lane == 0) sx = 0.0;
                const double vin = pbase + sc, vex = pbase + sx;
                int cand = INT_MAX;
                if (!take_last && vin > t_in && !(vex > t_in)) {
                    double run = vex;
#pragma unroll
                    for (int k = 0; k < kVec; ++k) {
                        run += (double)r[k];
                        if (cand == INT_MAX && run > t_in && r[k] > 0.f) cand = e0 + iv * kVec + k;
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) cand = min(cand, __shfl_xor_sync(0xffffffffu, cand, o));
                if (tok < 0 && cand != INT_MAX) tok = cand;
                pbase = __shfl_sync(0xffffffffu, vin, 31);
            }
            if (tok < 0) {                                    // u * R at or beyond the recomputed mass of the piece
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) lastel = max(lastel, __shfl_xor_sync(0xffffffffu, lastel, o));
                tok = lastel;
            }
        }
    }
    if (tok < 0) {
        // [P - Q]_+ has no mass (P == Q up to rounding) or a statistic is not finite: sample from
        // the target distribution of the same row.  Rare; one warp walks the row twice.
        bits |= f.bonus ? BS_DEV_NONFINITE : BS_DEV_RESIDUAL_FALLBACK;
        MassFn fp = f;
        fp.bonus = true;
        const int nv = p.V / kVec;
        double tot = 0.0;
        for (int v0 = 0; v0 < nv; v0 += 32) {
            float vs = 0.f;
            if (v0 + lane < nv) {
                const uint4 a = __ldcg(reinterpret_cast<const uint4*>(tp) + v0 + lane);
                float r[kVec];
                RsElems<T>::masses(a, a, fp, r);
#pragma unroll
                for (int k = 0; k < kVec; ++k) vs += r[k];
            }
            tot += __shfl_sync(0xffffffffu, warp_scan_incl((double)vs), 31);
        }
        if (tot > 0.0 && isfinite(tot)) {
            const double target = (double)u * tot;
            double base = 0.0;
            int lastel = -1;
            for (int v0 = 0; v0 < nv && tok < 0; v0 += 32) {
                float r[kVec];
#pragma unroll
                for (int k = 0; k < kVec; ++k) r[k] = 0.f;
                if (v0 + lane < nv) {
                    const uint4 a = __ldcg(reinterpret_cast<const uint4*>(tp) + v0 + lane);
                    RsElems<T>::masses(a, a, fp, r);
                }
                float vs = 0.f;
#pragma unroll
                for (int k = 0; k < kVec; ++k) {
                    vs += r[k];
                    if (r[k] > 0.f) lastel = (v0 + lane) * kVec + k;
                }
                const double sc = warp_scan_incl((double)vs);
                double sx = __shfl_up_sync(0xffffffffu, sc, 1);
                if (lane == 0) sx = 0.0;
                const double vin = base + sc, vex = base + sx;
                int cand = INT_MAX;
                if (vin > target && !(vex > target)) {
                    double run = vex;
#pragma unroll
                    for (int k = 0; k < kVec; ++k) {
                        run += (double)r[k];
                        if (cand == INT_MAX && run > target && r[k] > 0.f) cand = (v0 + lane) * kVec + k;
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) cand = min(cand, __shfl_xor_sync(0xffffffffu, cand, o));
                if (cand != INT_MAX) tok = cand;
                base = __shfl_sync(0xffffffffu, vin, 31);
            }
            if (tok < 0) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) lastel = max(lastel, __shfl_xor_sync(0xffffffffu, lastel, o));
                tok = lastel;
            }
        }
        if (tok < 0) { tok = 0; bits |= BS_DEV_NONFINITE; }
    }
    if (p.mode == kResidDraft) {                              // drafting: the token is the whole output
        if (lane == 0) {
            p.draft_out[(size_t)b * p.Gmax + p.position] = tok;
            // the status word belongs to the verification call that follows (it assigns it): what the
            // drafting pass found travels in the spare bit of the word of drafted positions
            if (bits) atomicOr(p.draft_ready + b, 0x80000000u);
            p.ticket[b] = 0u;
        }
        return;
    }
    // ---- outputs: the tau accepted drafts, the sampled token, padding ----
    int32_t* ot = p.out_tokens + (size_t)b * (p.Gmax + 1);
    for (int j = lane; j <= p.Gmax; j += 32)
        ot[j] = j < sq.tau ? p.tokens[(size_t)b * p.Gmax + j] : (j == sq.tau ? tok : -1);
    if (lane == 0) {
        p.out_len[b] = sq.tau + 1;
        if (bits) p.status[b] |= bits;
        p.ticket[b] = 0u;                                     // leave the counter clear for the next call
    }
}

}  // namespace bs
