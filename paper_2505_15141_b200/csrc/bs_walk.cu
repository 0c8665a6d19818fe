// bs_verify_walk: Algorithm 6 from its second line on, in one launch and in the algorithm's own
// order -- position after position, stopping at the first rejection ("break"), so the rows behind
// the first rejected draft are never read.
//
// Every sequence is shared by a fixed group of nG CTAs (up to 8), and every CTA holds a share of
// several sequences and interleaves them, so that a sequence with a long run of accepted drafts
// keeps a slice of many CTAs busy rather than one CTA alone.  For position k the group streams
// target row k and draft row k (bulk async copies into a ring of 32 KB stages, 16 consumer warps,
// online softmax: the pipeline of the row-statistics kernel), every CTA its contiguous share of
// the 2 * nseg segments (greedy mode: target rows only, arg-max instead of the statistics).  A finisher warp per CTA publishes the
// pieces and counts them on the sequence's ticket; the finisher that completes position k merges
// the two rows, tests r <= min{1, P/Q} for the drafted token and publishes the decision word of
// the sequence.  The producers of the group wait for that word (bounded), then stream position
// k + 1, or -- at the first rejection, or after the bonus row when everything passed -- the row
// pair of the stop position again (it has just been read: partly still in L2) for the residual
// masses; the finisher that completes that count runs the inverse CDF (level 2 of the resampling
// kernel).  In greedy mode the deciding finisher emits the arg-max of the stop row itself and the
// shares only acknowledge the decision, so that the last one can clear the sequence's words.
//
// CTAs of one group wait for one another, so the kernel is launched cooperatively (all CTAs
// resident).  Every wait is bounded; a wait that gives up sets the abort word and the CTA drains.
#include <atomic>
#include "bs_walk_common.cuh"

namespace bs {

// Per event handed to the finisher (written by consumer warp 0).
struct WkEvent {
    int type, b, k, row, first_sg, last_sg;
};
// A sequence in the producer's table: its share, the position it is at, and what it is waiting for.
struct WkSeq {
    int b, part, k, g;
    int stage;             // 0: position k to be streamed, 1: waiting for its decision, 2: done
};
constexpr int kWkMaxSeqs = 32;

// Stats items counted on the sequence's ticket once position k is complete.
template <bool GREEDY>
__device__ __forceinline__ unsigned wk_cum(int k, int g, int nseg) {
    if (GREEDY) return (unsigned)(nseg * (k + 1));           // target rows only
    return k < g ? (unsigned)(2 * nseg * (k + 1)) : (unsigned)(2 * nseg * g + nseg);
}
__device__ __forceinline__ unsigned ld_volatile_u32(const uint32_t* p) {
    return *reinterpret_cast<const volatile uint32_t*>(p);
}

template <typename T, bool GREEDY>
__global__ void __launch_bounds__(kWkThreads, 2) verify_walk_kernel(const WalkParams p) {
    extern __shared__ __align__(128) unsigned char ring[];    // kWkStages * 32 KB
    __shared__ __align__(8) unsigned long long s_full[kWkStages];
    __shared__ __align__(8) unsigned long long s_empty[kWkStages];
    __shared__ __align__(8) unsigned long long s_evbar[kWkRing];
    __shared__ __align__(8) unsigned long long s_evfree[kWkRing];
    __shared__ WkMeta s_meta[kWkStages];
    __shared__ WkEvent s_ev[kWkRing];
    __shared__ float2 s_red[kWkRing][kWkWarps];
    __shared__ float2 s_fin[2];
    __shared__ WkSeq s_seq[kWkMaxSeqs];

    const VerifyParams& v = p.v;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kVec = Elem<T>::kVec;

    if (tid == 0) {
        for (int s = 0; s < kWkStages; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), kWkWarps);
        }
        for (int s = 0; s < kWkRing; ++s) {
            mbar_init(smem_u32(&s_evbar[s]), kWkWarps);
            mbar_init(smem_u32(&s_evfree[s]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_enter();                                              // gamma comes from the kernel before this one

    if (warp == kWkWarps) {
        // =============================== producer ===============================
        // This CTA holds one share (part of nG) of several sequences: pair q = b * nG + part belongs
        // to CTA q % gridDim.x.  The producer keeps all of them moving: it streams whatever is
        // ready and only sleeps when every one of its sequences is waiting for a decision.
        if (lane != 0) return;
        int slot = 0;
        uint32_t ph = 0;
        bool ok = true;
        // one stage: wait for the slot, write the record, arm the barrier, copy
        auto issue = [&](const WkMeta& m, const T* src0, const T* src1, uint32_t bytes) -> bool {
            if (!mbar_wait(smem_u32(&s_empty[slot]), ph ^ 1u)) return false;
            s_meta[slot] = m;
            const uint32_t bar = smem_u32(&s_full[slot]);
            const uint32_t dst = smem_u32(ring + (size_t)slot * kSegBytes);
            if (m.type == kItemEnd || m.type == kItemAck) {
                mbar_arrive(bar);                              // nothing to copy: the phase completes at once
            } else {
                mbar_arrive_expect_tx(bar, src1 ? 2u * bytes : bytes);
                bulk_load(dst, src0, bytes, bar);
                if (src1) bulk_load(dst + kResSegBytes, src1, bytes, bar);
            }
            if (++slot == kWkStages) { slot = 0; ph ^= 1u; }
            return true;
        };
        const int npairs = v.B * p.nG;
        int nmine = 0;
        for (int q = blockIdx.x; q < npairs && nmine < kWkMaxSeqs; q += gridDim.x) {
            const int b = q / p.nG;
            s_seq[nmine++] = WkSeq{b, q - b * p.nG, 0, clamp_gamma(v.gamma[b], v.Gmax), 0};
        }
        int alive = nmine;
        long long t_last = clock64();
        while (alive > 0 && ok) {
            bool progress = false;
            unsigned dd[8];                                   // decision words of eight shares, asked for together
            for (int si = 0; si < nmine && ok; ++si) {
                if ((si & 7) == 0) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dd[i] = (si + i < nmine && s_seq[si + i].stage == 1) ? ld_volatile_u32(p.dec + s_seq[si + i].b) : 0u;
                }
                WkSeq sq = s_seq[si];
                if (sq.stage == 2) continue;
                const int b = sq.b, g = sq.g, part = sq.part;
                if (sq.stage == 1) {
                    // ---- has position k been decided (by whichever finisher of the group completed it)? ----
                    unsigned d = 0u;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if ((si & 7) == i) d = dd[i];
                    if ((d >> 1) != (unsigned)(sq.k + 1)) continue;
                    __threadfence();
                    progress = true;
                    if (sq.k < g && (d & 1u)) {                // accepted: on to the next position
                        sq.k += 1;
                        sq.stage = 0;
                    } else {
                        if (GREEDY) {
                            // the deciding finisher has emitted the arg-max already; this share only
                            // reports that it has seen the decision, so that the words can be cleared
                            WkMeta m;
                            m.type = kItemAck; m.b = b; m.k = sq.k; m.row = 0; m.sg = 0; m.nvec = 0; m.flags = 3;
                            m.kt = m.kd = 0.f; m.at = m.ad = 1.f;
                            ok = issue(m, nullptr, nullptr, 0);
                            sq.stage = 2;
                            --alive;
                            s_seq[si] = sq;
                            continue;
                        }
                        // ---- stop at k: residual [P_k - Q_k]_+ (rejected) or the bonus row P_k (k == gamma) ----
                        const int k = sq.k;
                        const bool bonus = k >= g;
                        const T* tp = row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, k, v.V);
                        const T* dp = bonus ? nullptr : row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, k, v.V);
                        const float2 ts = __ldcg(v.row_stats + (size_t)b * v.R + k);
                        float kt, at, kd = 0.f, ad = 1.f;
                        MassFn::fold(ts.x, ts.y, v.c, kt, at);
                        if (!bonus) {
                            const float2 ds = __ldcg(v.row_stats + (size_t)b * v.R + v.Gmax + 1 + k);
                            MassFn::fold(ds.x, ds.y, v.c, kd, ad);
                        }
                        const int rseg = p.r.seg, rnseg = p.r.nseg;
                        const int j0 = (int)((long long)rnseg * part / p.nG), j1 = (int)((long long)rnseg * (part + 1) / p.nG);
                        for (int sg = j0; sg < j1 && ok; ++sg) {
                            const int e0 = sg * rseg;
                            const int n = min(rseg, v.V - e0);
                            WkMeta m;
                            m.type = kItemMass; m.b = b; m.k = k; m.row = bonus ? 1 : 0; m.sg = sg; m.nvec = n / kVec;
                            m.flags = (sg == j0 ? 1 : 0) | (sg == j1 - 1 ? 2 : 0);
                            m.kt = kt; m.kd = kd; m.at = at; m.ad = ad;
                            ok = issue(m, tp + e0, bonus ? nullptr : dp + e0, (uint32_t)n * (uint32_t)sizeof(T));
                        }
                        sq.stage = 2;                          // this sequence is done for the producer
                        --alive;
                        s_seq[si] = sq;
                        continue;
                    }
                }
                // ---- position k: this CTA's share of target row k and, below gamma, draft row k ----
                {
                    const int k = sq.k;
                    const int nrows = (!GREEDY && !p.drafted && k < g) ? 2 : 1;
                    const int items = nrows * v.nseg;
                    const int i0 = (int)((long long)items * part / p.nG), i1 = (int)((long long)items * (part + 1) / p.nG);
                    for (int i = i0; i < i1 && ok; ++i) {
                        const int row = i / v.nseg, sg = i - row * v.nseg;
                        const T* rowp = row == 0 ? row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, k, v.V)
                                                 : row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, k, v.V);
                        const int e0 = sg * v.seg;
                        const int n = min(v.seg, v.V - e0);
                        WkMeta m;
                        m.type = kItemStats; m.b = b; m.k = k; m.row = row; m.sg = sg; m.nvec = n / kVec;
                        m.flags = ((sg == 0 || i == i0) ? 1 : 0) | ((sg == v.nseg - 1 || i == i1 - 1) ? 2 : 0);
                        m.kt = m.kd = 0.f; m.at = m.ad = 1.f;
                        ok = issue(m, rowp + e0, nullptr, (uint32_t)n * (uint32_t)sizeof(T));
                    }
                    sq.stage = 1;
                    s_seq[si] = sq;
                    progress = true;
                }
            }
            if (progress) {
                t_last = clock64();
            } else {
                if (clock64() - t_last > kWaitCycles) ok = false;
                __nanosleep(64);
            }
        }
        if (!ok) atomicExch(v.abort_flag, 1);
        // the end marker lets the consumers and the finisher leave (also after a failed wait, if a slot frees up)
        WkMeta e;
        e.type = kItemEnd; e.b = 0; e.k = 0; e.row = 0; e.sg = 0; e.nvec = 0; e.flags = 2; e.kt = e.kd = 0.f; e.at = e.ad = 1.f;
        issue(e, nullptr, nullptr, 0);
        return;
    }

    if (warp == kWkWarps + 1) {
        // =============================== finisher ===============================
        for (int ev = 0;; ++ev) {
            const int rs = ev % kWkRing;
            if (!mbar_wait_warp(smem_u32(&s_evbar[rs]), (uint32_t)(ev / kWkRing) & 1u)) {
                if (lane == 0) atomicExch(v.abort_flag, 1);
                return;
            }
            const WkEvent e = s_ev[rs];
            float2 mine = make_float2(-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f);
            if (lane < kWkWarps) mine = s_red[rs][lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_evfree[rs]));   // the slot may be reused
            if (e.type == kItemEnd) return;
            const int b = e.b, k = e.k;
            const int graw = v.gamma[b];
            const int g = clamp_gamma(graw, v.Gmax);
            const int len = e.last_sg - e.first_sg + 1;

            if (e.type == kItemAck) {
                // ---- greedy: one more share has seen the stop decision; the last one clears the words ----
                unsigned old = 0;
                if (lane == 0) old = atomicAdd(p.r.ticket + b, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old + 1u == (unsigned)p.nG && lane == 0) {
                    p.r.ticket[b] = 0u;
                    v.ticket[b] = 0u;
                    p.dec[b] = 0u;
                }
                continue;
            }
            if (GREEDY && e.type == kItemStats) {
                // ---- a piece of target row k: (max, arg-max); the drafted token passes iff it is the arg-max ----
                ArgMax a = warp_best(ArgMax{mine.x, __float_as_int(mine.y)});
                float2* pp = v.partial + ((size_t)b * v.R + k) * v.S;
                for (int q = e.first_sg + lane; q <= e.last_sg; q += 32)
                    pp[q] = (q == e.first_sg) ? make_float2(a.m, __int_as_float(a.idx))
                                              : make_float2(-INFINITY, __int_as_float(INT_MAX));
                int x = 0;
                if (k < g) x = v.tokens[(size_t)b * v.Gmax + k];
                __threadfence();
                __syncwarp();
                unsigned old = 0;
                if (lane == 0) old = atomicAdd(v.ticket + b, (unsigned)len);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old + (unsigned)len != wk_cum<true>(k, g, v.nseg)) continue;
                __threadfence();
                ArgMax best{-INFINITY, INT_MAX};
                for (int q = lane; q < v.nseg; q += 32) {
                    const float2 t = __ldcg(pp + q);
                    best = better(best, ArgMax{t.x, __float_as_int(t.y)});
                }
                best = warp_best(best);
                if (best.idx == INT_MAX) best.idx = 0;        // row of -inf / NaN only
                const bool bad = k < g && (x < 0 || x >= v.V);
                const bool acc = k < g && !bad && x == best.idx;
                int bits = (k == 0 && graw != g) ? BS_DEV_BAD_GAMMA : 0;
                if (bad) bits |= BS_DEV_BAD_TOKEN;
                if (lane == 0) {
                    v.row_stats[(size_t)b * v.R + k] = make_float2(best.m, __int_as_float(best.idx));
                    if (k == 0) v.status[b] = bits; else if (bits) atomicOr(v.status + b, bits);
                }
                if (!acc) {
                    // stop at k: the emitted token is the arg-max of target row k (Section 2, temperature 0)
                    int32_t* ot = p.r.out_tokens + (size_t)b * (v.Gmax + 1);
                    for (int j = lane; j <= v.Gmax; j += 32)
                        ot[j] = j < k ? v.tokens[(size_t)b * v.Gmax + j] : (j == k ? best.idx : -1);
                    for (int j = lane; j < v.Gmax; j += 32) {
                        if (v.p_tok) v.p_tok[(size_t)b * v.Gmax + j] = 0.f;
                        if (v.q_tok) v.q_tok[(size_t)b * v.Gmax + j] = 0.f;
                    }
                    if (lane == 0) {
                        v.accept_len[b] = k;
                        p.r.out_len[b] = k + 1;
                    }
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicExch(p.dec + b, ((unsigned)(k + 1) << 1) | (acc ? 1u : 0u));
                continue;
            }

            if (e.type == kItemStats) {
                // ---- a piece of target row k (row 0) or draft row k (row 1) ----
                const float2 out = warp_merge(Online{mine.x, mine.y}, v.c);
                const int slot_r = e.row == 0 ? k : v.Gmax + 1 + k;
                float2* pp = v.partial + ((size_t)b * v.R + slot_r) * v.S;
                for (int q = e.first_sg + lane; q <= e.last_sg; q += 32)
                    pp[q] = (q == e.first_sg) ? out : make_float2(-INFINITY, 0.f);
                __threadfence();
                __syncwarp();
                unsigned old = 0;
                if (lane == 0) old = atomicAdd(v.ticket + b, (unsigned)len);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old + (unsigned)len != (p.drafted ? wk_cum<true>(k, g, v.nseg) : wk_cum<false>(k, g, v.nseg))) continue;
                // ---- position k is complete: merge its rows (lanes 0..15: target, 16..31: draft), decide ----
                // Everything the decision needs is asked for in two rounds of independent loads: the drafted
                // token, the uniform and all partial slots of the two rows, then the two logits at the token
                // (a load that waits for another costs a full trip through a busy memory system; the fence
                // above would have waited for any of them issued earlier).
                __threadfence();
                int x = 0;
                float tl = 0.f, dl = 0.f, u = 2.f;
                bool bad = false;
                if (k < g) {
                    x = v.tokens[(size_t)b * v.Gmax + k];
                    u = v.u_accept[(size_t)b * v.Gmax + k];
                }
                {
                    const int half = lane >> 4, hl = lane & 15;
                    const int rr = half == 0 ? k : v.Gmax + 1 + k;
                    const bool mine_row = half == 0 || (k < g && !p.drafted);
                    const float2* qq = v.partial + ((size_t)b * v.R + rr) * v.S;
                    Online o{-INFINITY, 0.f};
                    for (int q0 = hl; q0 < v.nseg; q0 += 64) {        // four slots per lane in flight
                        float2 t[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int q = q0 + 16 * i;
                            t[i] = (mine_row && q < v.nseg) ? __ldcg(qq + q) : make_float2(-INFINITY, 0.f);
                        }
                        if (q0 == hl && k < g) {                      // the token has arrived by now: its two logits
                            bad = x < 0 || x >= v.V;
                            if (!bad) {
                                tl = Elem<T>::load(row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, k, v.V) + x);
                                dl = Elem<T>::load(row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, k, v.V) + x);
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) o.merge(t[i].x, t[i].y, v.c);
                    }
                    // lanes whose first slot lies beyond the row never entered the loop: lane 0 always did
                    tl = __shfl_sync(0xffffffffu, tl, 0);
                    dl = __shfl_sync(0xffffffffu, dl, 0);
                    bad = __shfl_sync(0xffffffffu, (int)bad, 0) != 0;
                    float M = o.m;
#pragma unroll
                    for (int off = 8; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
                    float Z = o.s * rescale(o.m, M, v.c);
#pragma unroll
                    for (int off = 8; off > 0; off >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, off);
                    if (hl == 0 && mine_row) {
                        s_fin[half] = make_float2(M, Z);
                        v.row_stats[(size_t)b * v.R + rr] = make_float2(M, Z);
                    }
                }
                __syncwarp();
                const float2 ts = s_fin[0];
                int bits = (k == 0 && graw != g) ? BS_DEV_BAD_GAMMA : 0;
                bool missing = false;                          // drafted mode: position k was never drafted
                if (p.drafted && k < g) {
                    if (lane == 0) s_fin[1] = __ldcg(v.row_stats + (size_t)b * v.R + v.Gmax + 1 + k);
                    const unsigned ready = __ldcg(v.draft_ready + b);
                    missing = ((ready >> k) & 1u) == 0u;
                    if (missing) bits |= BS_DEV_DRAFT_MISSING;
                    if (ready >> 31) bits |= BS_DEV_NONFINITE;   // a drafting pass could not sample its row
                    __syncwarp();
                }
                if (!(ts.y > 0.f) || !isfinite(ts.y) || !isfinite(ts.x)) bits |= BS_DEV_NONFINITE;
                bool acc = false;
                float pj = 0.f, qj = 0.f;
                if (k < g) {
                    const float2 ds = s_fin[1];
                    if (!(ds.y > 0.f) || !isfinite(ds.y) || !isfinite(ds.x)) bits |= BS_DEV_NONFINITE;
                    if (bad) {
                        bits |= BS_DEV_BAD_TOKEN;
                    } else if (!missing) {
                        // log2 of the two probabilities; the ratio is formed in the log domain
                        const float lp = (tl - ts.x) * v.c - log2f(ts.y);
                        const float lq = (dl - ds.x) * v.c - log2f(ds.y);
                        pj = exp2f(lp);
                        qj = exp2f(lq);
                        // r <= min{1, P/Q}; Q(x) = 0 counts as an infinite ratio
                        acc = (lq == -INFINITY) ? true : (u <= fminf(1.f, exp2f(lp - lq)));
                    }
                }
                if (lane == 0) {
                    if (k < g) {
                        if (v.p_tok) v.p_tok[(size_t)b * v.Gmax + k] = pj;
                        if (v.q_tok) v.q_tok[(size_t)b * v.Gmax + k] = qj;
                    }
                    if (k == 0) v.status[b] = bits; else if (bits) atomicOr(v.status + b, bits);
                    if (!acc) v.accept_len[b] = k;             // first rejection, or k == gamma: everything passed
                }
                if (!acc) {                                    // positions behind the stop were not looked at
                    for (int j = (k < g ? k + 1 : k) + lane; j < v.Gmax; j += 32) {
                        if (v.p_tok) v.p_tok[(size_t)b * v.Gmax + j] = 0.f;
                        if (v.q_tok) v.q_tok[(size_t)b * v.Gmax + j] = 0.f;
                    }
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicExch(p.dec + b, ((unsigned)(k + 1) << 1) | (acc ? 1u : 0u));
                if (acc && k + 1 < g && lane == 0) {
                    // the walk goes on: ask L2 for the two logits the next decision will need (nobody waits for this)
                    const int xn = v.tokens[(size_t)b * v.Gmax + k + 1];
                    if (xn >= 0 && xn < v.V) {
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, k + 1, v.V) + xn));
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, k + 1, v.V) + xn));
                    }
                }
            } else {
                // ---- this CTA's share of the residual masses of the stop position k is written ----
                __threadfence();
                unsigned old = 0;
                if (lane == 0) old = atomicAdd(p.r.ticket + b, (unsigned)len);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old + (unsigned)len != (unsigned)p.r.nseg) continue;
                __threadfence();
                RsSeq sq;
                sq.tau = k; sq.bonus = k >= g; sq.wgt = sq.bonus ? 1 : 2;
                MassFn f;
                f.c = v.c; f.bonus = sq.bonus != 0;
                const float2 ts = __ldcg(v.row_stats + (size_t)b * v.R + k);
                MassFn::fold(ts.x, ts.y, v.c, f.kt, f.at);
                f.kd = 0.f; f.ad = 1.f;
                if (!f.bonus) {
                    const float2 ds = __ldcg(v.row_stats + (size_t)b * v.R + v.Gmax + 1 + k);
                    MassFn::fold(ds.x, ds.y, v.c, f.kd, f.ad);
                }
                rs_level2<T>(p.r, b, sq, f);                   // token, out_tokens, out_len; clears the mass ticket
                if (lane == 0) {                               // leave the workspace clean for the next call
                    v.ticket[b] = 0u;
                    p.dec[b] = 0u;
                    if (p.drafted) v.draft_ready[b] = 0u;      // consumed: a later round must draft again
                }
            }
        }
    }

    // ================================= consumers =================================
    Online on{-INFINITY, 0.f};
    ArgMax am{-INFINITY, INT_MAX};
    int first_sg = 0;
    int ev = 0;                                               // events posted by this CTA
    int slot = 0;
    uint32_t ph = 0;
    for (;;) {
        if (!mbar_wait_warp(smem_u32(&s_full[slot]), ph)) { atomicExch(v.abort_flag, 1); return; }
        const WkMeta m = s_meta[slot];
        const uint32_t base = smem_u32(ring + (size_t)slot * kSegBytes);
        if (m.flags & 1) first_sg = m.sg;
        float2 wr = make_float2(-INFINITY, 0.f);
        if (m.type == kItemStats) {
            // one 32 KB segment of one row: online softmax statistics, one exp per logit
            uint4 x[kWkVecPerThread];
#pragma unroll
            for (int q = 0; q < kWkVecPerThread; ++q)
                x[q] = (q * kWkConsumers + tid < m.nvec) ? lds128(base + (uint32_t)(q * kWkConsumers + tid) * 16u)
                                                         : neg_inf_vec<T>();
            fence_reads_before_refill();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
            if (GREEDY) {
                argmax_add<T, kWkVecPerThread>(am, x, m.sg * v.seg + tid * kVec, kWkConsumers * kVec);
                if (m.flags & 2) {
                    am = warp_best(am);
                    wr = make_float2(am.m, __int_as_float(am.idx));
                    am = ArgMax{-INFINITY, INT_MAX};
                }
            } else {
                online_add<T, kWkVecPerThread>(on, x, v.c);
                if (m.flags & 2) {
                    wr = warp_merge(on, v.c);
                    on = Online{-INFINITY, 0.f};
                }
            }
        } else if (m.type == kItemMass) {
            // a 16 KB segment of the row pair: warp w owns the w-th 1 KB piece and writes its mass
            MassFn f;
            f.c = v.c; f.kt = m.kt; f.kd = m.kd; f.at = m.at; f.ad = m.ad; f.bonus = m.row != 0;
            const uint32_t pb = base + (uint32_t)(warp * kRsPieceBytes + lane * 16);
            uint4 a[kRsVecPerLane], d[kRsVecPerLane];
            bool valid[kRsVecPerLane];
#pragma unroll
            for (int q = 0; q < kRsVecPerLane; ++q) {
                valid[q] = warp * kRsPieceVecs + q * 32 + lane < m.nvec;
                if (valid[q]) {
                    a[q] = lds128(pb + (uint32_t)(q * 512));
                    d[q] = f.bonus ? a[q] : lds128(pb + (uint32_t)(kResSegBytes + q * 512));
                }
            }
            fence_reads_before_refill();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
            float acc = 0.f;
#pragma unroll
            for (int q = 0; q < kRsVecPerLane; ++q) {
                if (valid[q]) {
                    float r[kVec];
                    RsElems<T>::masses(a[q], d[q], f, r);
                    float vs = 0.f;
#pragma unroll
                    for (int i = 0; i < kVec; ++i) vs += r[i];
                    acc += vs;
                }
            }
            acc = warp_sum(acc);
            if (lane == 0) {
                p.r.resid_partial[(size_t)m.b * p.r.S + m.sg * kRsWarps + warp] = acc;
                if (m.flags & 2) __threadfence();             // the share's masses are visible before the event
            }
        } else {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
        }
        if (++slot == kWkStages) { slot = 0; ph ^= 1u; }

        if (m.flags & 2) {
            // ---- end of a row piece / of the share / of the work: one event for the finisher ----
            const int rs = ev % kWkRing;
            if (ev >= kWkRing && !mbar_wait_warp(smem_u32(&s_evfree[rs]), (uint32_t)(ev / kWkRing - 1) & 1u)) {
                atomicExch(v.abort_flag, 1);
                return;
            }
            if (lane == 0) {
                s_red[rs][warp] = wr;
                if (warp == 0) s_ev[rs] = WkEvent{m.type, m.b, m.k, m.row, first_sg, m.sg};
                mbar_arrive(smem_u32(&s_evbar[rs]));          // release: the writes above are visible to the finisher
            }
            ++ev;
            if (m.type == kItemEnd) return;
        }
    }
}

static std::atomic<int> g_wk_blocks[4][64];        // resident CTAs per SM (0 = not queried)

template <typename T, bool GREEDY>
static bs_status launch_walk(WalkParams& p, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    const int variant = (Elem<T>::kDtype == BS_F32 ? 0 : 2) + (GREEDY ? 1 : 0);
    const size_t smem = (size_t)kWkStages * kSegBytes;
    if (!g_wk_blocks[variant][dev]) {
        if (cudaFuncSetAttribute(verify_walk_kernel<T, GREEDY>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return cuda_status(cudaGetLastError());
        int nb = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, verify_walk_kernel<T, GREEDY>, kWkThreads, smem) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        if (nb < 1) return BS_ERR_UNSUPPORTED;
        g_wk_blocks[variant][dev] = nb > 2 ? 2 : nb;
    }
    // groups of CTAs wait for one another: never more CTAs than can be resident together
    const int max_grid = g_wk_blocks[variant][dev] * sm_count();
    // every sequence is shared by nG CTAs and every CTA holds a share of about B * nG / grid sequences,
    // so a long run of accepted drafts keeps a slice of many CTAs busy instead of one whole CTA
    // (measured on 256 x 152064 fp32: 3.5 shares per CTA is the best trade between the time a
    // sequence waits for its CTAs' other work and the time it takes to stream a share)
    int nG = (int)((7LL * max_grid + p.v.B) / (2LL * p.v.B));
    if (nG > 8) nG = 8;
    if (nG > p.v.nseg) nG = p.v.nseg;                        // every CTA of a group gets a segment of every row
    if (nG < 1) nG = 1;
    while (nG > 1 && (long long)p.v.B * nG > (long long)max_grid * kWkMaxSeqs) --nG;
    p.nG = nG;
    const long long pairs = (long long)p.v.B * nG;
    const int grid = pairs < max_grid ? (int)pairs : max_grid;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kWkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set-up overlaps the previous kernel's drain
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    return cuda_status(cudaLaunchKernelEx(&cfg, verify_walk_kernel<T, GREEDY>, p));
}

}  // namespace bs

using namespace bs;

static bs_status run_walk(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                          const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                          const float* u_resample, float temperature, int B, int Gmax, int V,
                          int32_t* accept_len, float* p_tok, float* q_tok, int32_t* out_tokens,
                          int32_t* out_len, void* workspace, size_t workspace_bytes, void* stream, int drafted) {
    if (B < 1 || Gmax < 0 || V < 1) return BS_ERR_INVALID_ARG;
    if (B > BS_MAX_BATCH || Gmax > BS_MAX_GAMMA || V > BS_MAX_VOCAB) return BS_ERR_UNSUPPORTED;
    if (dtype != BS_F32 && dtype != BS_BF16) return BS_ERR_INVALID_ARG;
    if (!(temperature >= 0.f) || !isfinite(temperature)) return BS_ERR_INVALID_ARG;
    const bool greedy = temperature == 0.f;
    if (!target_logits || !gamma || !accept_len || !out_tokens || !out_len || !workspace) return BS_ERR_INVALID_ARG;
    if (Gmax > 0 && !draft_tokens) return BS_ERR_INVALID_ARG;
    if (!greedy && (!u_resample || (Gmax > 0 && (!draft_logits || !u_accept)))) return BS_ERR_INVALID_ARG;
    const size_t es = dtype == BS_F32 ? 4 : 2;
    if (((size_t)V * es) % 16 != 0 || (reinterpret_cast<uintptr_t>(target_logits) & 15) ||
        (reinterpret_cast<uintptr_t>(draft_logits) & 15))
        return BS_ERR_UNSUPPORTED;                           // rows must start on 16-byte boundaries
    const Workspace w = workspace_layout(B, Gmax, V);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) return BS_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    WalkParams p;
    VerifyParams& v = p.v;
    v.target = target_logits; v.draft = draft_logits; v.tokens = draft_tokens; v.gamma = gamma;
    v.u_accept = u_accept; v.accept_len = accept_len; v.p_tok = p_tok; v.q_tok = q_tok;
    v.ticket = reinterpret_cast<uint32_t*>(ws + w.off_ticket_verify);
    v.ticket_row = reinterpret_cast<uint32_t*>(ws + w.off_ticket_row);
    v.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    v.abort_flag = reinterpret_cast<int32_t*>(ws + w.off_abort);
    v.row_stats = reinterpret_cast<float2*>(ws + w.off_row_stats);
    v.partial = reinterpret_cast<float2*>(ws + w.off_partial);
    v.B = B; v.Gmax = Gmax; v.V = V; v.R = w.R; v.S = w.S;
    v.seg = seg_elems(dtype);
    v.nseg = div_up(V, v.seg);
    v.c = greedy ? 1.f : kLog2e / temperature;
    v.mode = kModeVerify; v.position = 0; v.draft_ready = v.ticket_row; v.draft_out = nullptr;
    ResidParams& r = p.r;
    r.target = target_logits; r.draft = draft_logits; r.tokens = draft_tokens; r.gamma = gamma;
    r.accept_len = accept_len; r.u_resample = u_resample; r.out_tokens = out_tokens; r.out_len = out_len;
    r.ticket = reinterpret_cast<uint32_t*>(ws + w.off_ticket_resid);
    r.status = v.status;
    r.abort_flag = v.abort_flag;
    r.row_stats = v.row_stats;
    r.resid_partial = reinterpret_cast<float*>(ws + w.off_resid_partial);
    r.B = B; r.Gmax = Gmax; r.V = V; r.R = w.R; r.S = w.Sr;
    r.seg = res_seg_elems(dtype);
    r.nseg = div_up(V, r.seg);
    r.c = v.c;
    r.mode = kResidVerify; r.position = 0; r.draft_out = nullptr; r.draft_ready = nullptr;
    // decision words: the second B words of the per-row counter slot (the first B mark drafted positions)
    p.dec = v.ticket_row + B;
    p.nG = 1;
    p.look = 0;
    p.drafted = (drafted && !greedy) ? 1 : 0;         // greedy rounds never read draft rows anyway
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // groups of 2, 4 or 8 CTAs as thread-block clusters (hand-offs through distributed shared memory); rows of a
    // single segment and batches too large for that leave one CTA per sequence: the kernel of this file
    bs_status s;
    if (greedy) s = dtype == BS_F32 ? launch_walk_cluster<float, true>(p, st) : launch_walk_cluster<__nv_bfloat16, true>(p, st);
    else s = dtype == BS_F32 ? launch_walk_cluster<float, false>(p, st) : launch_walk_cluster<__nv_bfloat16, false>(p, st);
    if (s != BS_ERR_UNSUPPORTED) return s;
    if (greedy) return dtype == BS_F32 ? launch_walk<float, true>(p, st) : launch_walk<__nv_bfloat16, true>(p, st);
    return dtype == BS_F32 ? launch_walk<float, false>(p, st) : launch_walk<__nv_bfloat16, false>(p, st);
}

extern "C" bs_status bs_verify_walk(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                    const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                    const float* u_resample, float temperature, int B, int Gmax, int V,
                                    int32_t* accept_len, float* p_tok, float* q_tok, int32_t* out_tokens,
                                    int32_t* out_len, void* workspace, size_t workspace_bytes, void* stream) {
    return run_walk(target_logits, draft_logits, dtype, draft_tokens, gamma, u_accept, u_resample, temperature, B, Gmax,
                    V, accept_len, p_tok, q_tok, out_tokens, out_len, workspace, workspace_bytes, stream, 0);
}

extern "C" bs_status bs_verify_walk_drafted(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                            const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                            const float* u_resample, float temperature, int B, int Gmax, int V,
                                            int32_t* accept_len, float* p_tok, float* q_tok, int32_t* out_tokens,
                                            int32_t* out_len, void* workspace, size_t workspace_bytes, void* stream) {
    return run_walk(target_logits, draft_logits, dtype, draft_tokens, gamma, u_accept, u_resample, temperature, B, Gmax,
                    V, accept_len, p_tok, q_tok, out_tokens, out_len, workspace, workspace_bytes, stream, 1);
}
