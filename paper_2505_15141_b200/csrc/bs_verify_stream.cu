// Pipelined row-statistics kernel of bs_softmax_verify for rows that start on 16-byte
// boundaries (V * sizeof(element) a multiple of 16): softmax with temperature (Section 2 of the
// paper) and the accept loop of Algorithm 6, followed -- inside the same launch -- by the first
// half of Algorithm 6's resampling step for every sequence whose accept loop is already done.
//
// The flat list of work items (one item = one 32 KB segment of one valid row, sequences in batch
// order; ragged gamma_b handled through a prefix sum over the batch) is handed out in chunks of a
// few consecutive items: every CTA starts with the chunk of its own index and takes the next free
// one from a counter in the workspace, so the grid moves through the batch as a front a few
// sequences wide and sequence b is complete after about (b + 1) / B of the launch.  The finisher
// whose piece completes a sequence runs its accept scan and publishes the stop row tau_b; from then
// on the residual masses r_v = [P(v) - Q(v)]_+ of that row pair (the bonus row alone when every
// draft passed) are work like any other: they are handed out in a few "mass chunks" per sequence,
// which the CTAs take in preference to new statistics chunks.  The row pair was streamed a few
// microseconds earlier, so those reads are L2 hits rather than a second trip to DRAM.  Nobody waits
// for another CTA: mass chunks that become ready after a CTA has run out of statistics chunks are
// simply left, and bs_residual_sample computes whatever is missing.
//
//   warp 16 (one lane) producer: decides what comes next (a ready mass chunk, else the next
//                      statistics chunk), and for each stage arms a "full" mbarrier with the byte
//                      count and issues one or two bulk async copies (TMA, no multicast)
//                      global -> shared into a ring of 32 KB slots.
//   warps 0..15        consumers: wait for the slot, read it with conflict-free 128-bit shared
//                      loads, release it through an "empty" mbarrier, then either update a
//                      per-thread online softmax state (chunk max first, then ONE exp per logit)
//                      or, on a mass stage, form the masses of the warp's 1 KB piece and write
//                      their sum.
//   warp 17            finisher: takes what the consumers finish (a small ring of per-warp results
//                      in shared memory): merges a row piece, publishes it and does what the piece
//                      completes; counts a finished mass chunk.  The consumers never leave the
//                      stream.
//
// The per-thread state lives across the segments of a row piece; it is reduced only when the row
// or the chunk ends.  Every piece is published as a partial and counted on one atomic ticket per
// sequence; the finisher whose piece completes the count merges all rows of the sequence (one lane
// per row) and runs the accept scan.  Piece boundaries depend on the item list alone, not on which
// CTA took which chunk, so every reduction has a fixed order.  All waits on mbarriers are bounded;
// a wait that gives up sets the abort word and the thread leaves.
#include "bs_verify_common.cuh"
#include "bs_residual_level2.cuh"
#include "bs_pipeline.cuh"

namespace bs {

constexpr int kConsumerWarps = 16;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kStreamThreads = kConsumers + 64;                   // + producer warp + finisher warp
constexpr int kVecPerStage = kSegBytes / 16;                     // 2048
constexpr int kVecPerThread = kVecPerStage / kConsumers;         // 4
constexpr int kMaxStages = 3;
constexpr int kRedSlots = 8;                                     // events the consumers may run ahead of the finisher
constexpr int kChunkItems = 4;                                   // items of the list handed out together
static_assert(kVecPerThread * kConsumers == kVecPerStage, "stage must divide evenly over the consumers");
static_assert(kSegBytes == kRsStageBytes && kConsumerWarps == kRsWarps,
              "a slot holds one statistics segment or one stage of the resampling kernel");

constexpr int kStStats = 0, kStMass = 1, kStEnd = 2;

// Per-stage record written by the producer.  kind = kSt* | flags << 4; flags bit 0: first stage of a
// row piece, bit 1: last stage of a row piece / of a mass chunk, bit 2 (mass): the target row alone
// (bonus token).  w1 = b | lr << 13 | sg << 19 (b < 2^13, lr < 2^6, sg < 2^8); for a mass stage lr = 0
// and sg is the first 16 KB segment in the slot.
struct StageMeta {
    int kind, w1;
    int nvec, nvec2;            // valid 16-byte vectors (mass stages: in the first / second half of the slot)
    float kt, kd, at, ad;       // mass stages: the constants of MassFn
};
// Per event handed to the finisher, written by consumer warp 0: kind as above (flags dropped), w1 of the
// last stage, first segment of the piece.
struct PieceMeta {
    int kind, w1, first_sg;
};
static_assert(BS_MAX_BATCH <= (1 << 13) && 2 * BS_MAX_GAMMA + 1 < (1 << 6) &&
              BS_MAX_VOCAB / (kSegBytes / 4) <= (1 << 8) && BS_MAX_VOCAB / kResSegElemsMin <= (1 << 8),
              "StageMeta packing");

template <typename T, bool GREEDY>
__global__ void __launch_bounds__(kStreamThreads, 2) verify_stream_kernel(const VerifyParams p, const int nstages) {
    extern __shared__ __align__(128) unsigned char smem[];
    // layout: [nstages * 32 KB ring][prefix (B+1) ints]
    unsigned char* ring = smem;
    int* s_prefix = reinterpret_cast<int*>(smem + (size_t)nstages * kSegBytes);
    __shared__ __align__(8) unsigned long long s_full[kMaxStages];
    __shared__ __align__(8) unsigned long long s_empty[kMaxStages];
    // one barrier pair per event slot: a warp may run several events ahead of another, so arrivals
    // of different events must never meet on one barrier
    __shared__ __align__(8) unsigned long long s_redbar[kRedSlots];
    __shared__ __align__(8) unsigned long long s_redfree[kRedSlots];
    __shared__ PieceMeta s_piece[kRedSlots];
    __shared__ float2 s_fin[2 * BS_MAX_GAMMA + 1];            // merged row statistics of the sequence being finished
    __shared__ __align__(16) StageMeta s_meta[kMaxStages];
    __shared__ float2 s_red[kRedSlots][kConsumerWarps];
    __shared__ int s_scan[kStreamThreads / 32];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kVec = Elem<T>::kVec;

    if (tid == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), kConsumerWarps);
        }
        for (int s = 0; s < kRedSlots; ++s) {
            mbar_init(smem_u32(&s_redbar[s]), kConsumerWarps);
            mbar_init(smem_u32(&s_redfree[s]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    pdl_enter();                                              // gamma comes from the kernel before this one

    // ---- prefix sum of work items over the batch (all threads, redundantly per CTA) ----
    {
        const int per = div_up(p.B, kStreamThreads);
        const int b0 = tid * per;
        int local = 0;
        for (int k = 0; k < per; ++k) {
            const int b = b0 + k;
            if (b < p.B) local += mode_rows<GREEDY>(p, clamp_gamma(p.gamma[b], p.Gmax)) * p.nseg;
        }
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_scan[warp] = incl;
        __syncthreads();
        int woff = 0;
        for (int w = 0; w < warp; ++w) woff += s_scan[w];
        int run = woff + incl - local;
        for (int k = 0; k < per; ++k) {
            const int b = b0 + k;
            if (b < p.B) {
                s_prefix[b] = run;
                run += mode_rows<GREEDY>(p, clamp_gamma(p.gamma[b], p.Gmax)) * p.nseg;
            }
        }
        if (tid == kStreamThreads - 1) s_prefix[p.B] = run;
        __syncthreads();                                      // also publishes the mbarrier inits
    }
    const int total = s_prefix[p.B];
    // The residual masses are only of use to a resampling call: not in greedy mode, not while drafting.
    const bool masses = !GREEDY && p.mode != kModeDraft;
    // Mass words written by this launch carry this tag; the last CTA to leave bumps the epoch.
    const uint32_t epoch0 = __ldcg(p.sched + kSchedEpoch);
    const uint32_t tag = epoch_tag(epoch0);

    if (warp == kConsumerWarps) {
        // =============================== producer ===============================
        if (lane != 0) return;
        const int nchunks = div_up(total, kChunkItems);
        const int C = mass_chunks(p.rnseg);
        int slot = 0;
        uint32_t ph = 0;
        // one stage: wait for the slot, write the record, arm the barrier, copy
        auto issue = [&](const StageMeta& m, const void* s0, uint32_t n0, const void* s1, uint32_t n1) -> bool {
            if (!mbar_wait(smem_u32(&s_empty[slot]), ph ^ 1u)) return false;
            s_meta[slot] = m;
            const uint32_t bar = smem_u32(&s_full[slot]);
            const uint32_t dst = smem_u32(ring + (size_t)slot * kSegBytes);
            if (n0 + n1 == 0u) {
                mbar_arrive(bar);                             // nothing to copy: the phase completes at once
            } else {
                mbar_arrive_expect_tx(bar, n0 + n1);          // releases the record to the waiters
                bulk_load(dst, s0, n0, bar);
                if (n1) bulk_load(dst + kResSegBytes, s1, n1, bar);
            }
            if (++slot == nstages) { slot = 0; ph ^= 1u; }
            return true;
        };
        // chunk c of the item list
        auto stats_chunk = [&](int c) -> bool {
            const int lo = c * kChunkItems, hi = min(total, lo + kChunkItems);
            int b, lr, sg, g, rows_b;
            {
                int l = 0, h = p.B;                           // largest b with prefix[b] <= lo
                while (h - l > 1) {
                    const int mid = (l + h) >> 1;
                    if (s_prefix[mid] <= lo) l = mid; else h = mid;
                }
                b = l;
                const int local = lo - s_prefix[b];
                lr = local / p.nseg;
                sg = local - lr * p.nseg;
                g = clamp_gamma(p.gamma[b], p.Gmax);
                rows_b = mode_rows<GREEDY>(p, g);
            }
            for (int k = lo; k < hi; ++k) {
                const T* rowp = mode_row<T>(p, b, lr, g);
                const int e0 = sg * p.seg;
                const int n = min(p.seg, p.V - e0);
                const int flags = ((sg == 0 || k == lo) ? 1 : 0) | ((sg == p.nseg - 1 || k == hi - 1) ? 2 : 0);
                StageMeta m;
                m.kind = kStStats | (flags << 4);
                m.w1 = b | (lr << 13) | (sg << 19);
                m.nvec = n / kVec; m.nvec2 = 0;
                m.kt = m.kd = 0.f; m.at = m.ad = 1.f;
                if (!issue(m, rowp + e0, (uint32_t)n * (uint32_t)sizeof(T), nullptr, 0u)) return false;
                if (++sg == p.nseg) {                         // advance to the next item
                    sg = 0;
                    if (++lr == rows_b) {
                        lr = 0;
                        do {                                  // next sequence that contributes rows
                            ++b;
                            if (b < p.B) {
                                g = clamp_gamma(p.gamma[b], p.Gmax);
                                rows_b = mode_rows<GREEDY>(p, g);
                            }
                        } while (b < p.B && rows_b == 0);
                    }
                }
            }
            return true;
        };
        // The next mass chunk, if its sequence has been through the accept scan.  Chunks are taken in
        // order (chunk h = part h % C of sequence h / C); sequences complete nearly in batch order, so a
        // chunk is rarely held up behind a sequence that is late.  0: nothing ready, 1: done, -1: a wait gave up.
        auto mass_chunk = [&]() -> int {
            const uint32_t h = *reinterpret_cast<volatile uint32_t*>(p.sched + kSchedMassHead);
            const int b = (int)(h / (uint32_t)C);
            if (b >= p.B) return 0;
            const uint32_t mt = *reinterpret_cast<volatile uint32_t*>(p.mass_tau + b);
            if ((mt >> 8) != tag) return 0;
            if (atomicCAS(p.sched + kSchedMassHead, h, h + 1u) != h) return 0;   // another CTA took it
            __threadfence();                                  // the row statistics were written before the word
            const int part = (int)(h - (uint32_t)b * (uint32_t)C);
            const int tau = (int)(mt & 0xffu) - 1;
            const int g = clamp_gamma(p.gamma[b], p.Gmax);
            const bool bonus = tau >= g;
            const int nit = rs_row_items(bonus, p.rnseg);
            const int i0 = (int)((long long)nit * part / C), i1 = (int)((long long)nit * (part + 1) / C);
            const float2 ts = __ldcg(p.row_stats + (size_t)b * p.R + tau);
            StageMeta m;
            m.kd = 0.f; m.ad = 1.f;
            MassFn::fold(ts.x, ts.y, p.c, m.kt, m.at);
            const T* tp = row_ptr(static_cast<const T*>(p.target), b, p.Gmax + 1, tau, p.V);
            const T* dp = tp;
            if (!bonus) {
                const float2 ds = __ldcg(p.row_stats + (size_t)b * p.R + p.Gmax + 1 + tau);
                MassFn::fold(ds.x, ds.y, p.c, m.kd, m.ad);
                dp = row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, tau, p.V);
            }
            for (int it = i0; it < i1; ++it) {
                const int sg = bonus ? 2 * it : it;           // a row sampled alone fills the slot with two segments
                const int e0 = sg * p.rseg;
                const int n = min(p.rseg, p.V - e0);
                const int n2 = !bonus ? n : (sg + 1 < p.rnseg ? min(p.rseg, p.V - e0 - p.rseg) : 0);
                m.kind = kStMass | (((it == i1 - 1 ? 2 : 0) | (bonus ? 4 : 0)) << 4);
                m.w1 = b | (sg << 19);
                m.nvec = n / kVec; m.nvec2 = n2 / kVec;
                if (!issue(m, tp + e0, (uint32_t)n * (uint32_t)sizeof(T), (bonus ? tp + p.rseg : dp) + e0,
                           (uint32_t)n2 * (uint32_t)sizeof(T)))
                    return -1;
            }
            return 1;
        };

        // Every CTA starts with the chunk of its own index; further chunks come from the counter, asked
        // for one ahead so that the answer has arrived by the time it is needed.
        int cur = (int)blockIdx.x < nchunks ? (int)blockIdx.x : -1;
        bool have_next = nchunks > (int)gridDim.x;
        unsigned next_raw = 0u;
        if (have_next) next_raw = atomicAdd(p.sched + kSchedCursor, 1u);
        bool ok = true, first = true;
        int tail = 1;                                         // mass chunks taken once the statistics chunks are gone
        while (ok) {
            if (masses && !first && (cur >= 0 || tail > 0)) {
                const int r = mass_chunk();
                if (r < 0) { ok = false; break; }
                if (r > 0) {
                    if (cur < 0) --tail;
                    continue;
                }
            }
            first = false;
            if (cur < 0) break;
            ok = stats_chunk(cur);
            cur = -1;
            if (have_next) {
                const int c = (int)gridDim.x + (int)next_raw;
                if (c < nchunks) {
                    cur = c;
                    next_raw = atomicAdd(p.sched + kSchedCursor, 1u);
                } else {
                    have_next = false;
                }
            }
        }
        if (!ok) { atomicExch(p.abort_flag, 1); return; }
        StageMeta e;
        e.kind = kStEnd | (2 << 4); e.w1 = 0; e.nvec = e.nvec2 = 0; e.kt = e.kd = 0.f; e.at = e.ad = 1.f;
        if (!issue(e, nullptr, 0u, nullptr, 0u)) atomicExch(p.abort_flag, 1);
        return;
    }

    if (warp == kConsumerWarps + 1) {
        // =============================== finisher ===============================
        // Takes the events the consumers post, in order.  A row piece: merge the 16 warp results,
        // publish the piece, and do whatever the piece completes (row merge, accept scan, hand the
        // stop row over to the mass chunks).  A mass chunk: count it.  The consumers never wait for
        // any of this.
        for (int pc = 0;; ++pc) {
            const int rs = pc % kRedSlots;
            if (!mbar_wait_warp(smem_u32(&s_redbar[rs]), (uint32_t)(pc / kRedSlots) & 1u)) {
                if (lane == 0) atomicExch(p.abort_flag, 1);
                return;
            }
            const PieceMeta pm = s_piece[rs];
            float2 mine = make_float2(-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f);
            if (lane < kConsumerWarps) mine = s_red[rs][lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_redfree[rs]));   // the slot may be reused
            if (pm.kind == kStEnd) break;
            const int m_b = pm.w1 & 0x1fff, m_lr = (pm.w1 >> 13) & 0x3f, m_sg = (pm.w1 >> 19) & 0xff;
            if (pm.kind == kStMass) {
                // every consumer warp has written the masses of its pieces of this chunk
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(p.mass_done + m_b, 1u);
                }
                continue;
            }
            float2 out;
            if (GREEDY) {
                ArgMax a = warp_best(ArgMax{mine.x, __float_as_int(mine.y)});
                out = make_float2(a.m, __int_as_float(a.idx));
            } else {
                out = warp_merge(Online{mine.x, mine.y}, p.c);
            }
            // ---- publish the piece; the finisher that completes the sequence does the rest ----
            const int first_sg = pm.first_sg;
            const int graw = p.gamma[m_b];
            const int gb = clamp_gamma(graw, p.Gmax);
            const int r = mode_slot(p, m_lr, gb);
            const int piece_len = m_sg - first_sg + 1;
            const int rows_mb = mode_rows<GREEDY>(p, gb);
            {
                float2* pp = p.partial + ((size_t)m_b * p.R + r) * p.S;
                // slot of the piece's first segment carries the result, the rest are neutral
                for (int q = first_sg + lane; q <= m_sg; q += 32)
                    pp[q] = (q == first_sg) ? out : make_float2(-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f);
            }
            // the loads of the accept test do not depend on the statistics: start them now, so
            // that they travel while the arrival counter does
            AcceptLoads al{0, 0.f, 0.f, 2.f, 0};
            if (p.mode != kModeDraft) al = accept_prefetch<T, GREEDY>(p, m_b, gb);
            __threadfence();
            __syncwarp();
            unsigned old = 0;
            if (lane == 0) old = atomicAdd(p.ticket + m_b, (unsigned)piece_len);
            old = __shfl_sync(0xffffffffu, old, 0);
            if (old + (unsigned)piece_len != (unsigned)(rows_mb * p.nseg)) continue;
            // ---- last piece of the sequence: merge every row (one lane per row), accept scan ----
            __threadfence();
            for (int lr0 = 0; lr0 < rows_mb; lr0 += 32) {
                const int lr = lr0 + lane;
                if (lr < rows_mb) {
                    const int rr = mode_slot(p, lr, gb);
                    const float2* pp = p.partial + ((size_t)m_b * p.R + rr) * p.S;
                    float2 st;
                    if (GREEDY) {
                        ArgMax a{-INFINITY, INT_MAX};
#pragma unroll 4
                        for (int q = 0; q < p.nseg; ++q) {
                            const float2 v = __ldcg(pp + q);
                            a = better(a, ArgMax{v.x, __float_as_int(v.y)});
                        }
                        if (a.idx == INT_MAX) a.idx = 0;      // row of -inf / NaN only
                        st = make_float2(a.m, __int_as_float(a.idx));
                    } else {
                        Online o{-INFINITY, 0.f};
#pragma unroll 4
                        for (int q = 0; q < p.nseg; ++q) {
                            const float2 v = __ldcg(pp + q);
                            o.merge(v.x, v.y, p.c);
                        }
                        st = make_float2(o.m, o.s);
                    }
                    s_fin[rr] = st;
                    p.row_stats[(size_t)m_b * p.R + rr] = st;
                }
            }
            __syncwarp();
            int tau = 0;
            if (p.mode == kModeDraft) {
                // the draft row's statistics are in place; greedy drafting ends here
                if (lane == 0) {
                    if (GREEDY) p.draft_out[(size_t)m_b * p.Gmax + p.position] = __float_as_int(s_fin[r].y);
                    __threadfence();
                    atomicOr(p.draft_ready + m_b, 1u << p.position);
                }
            } else if (p.mode == kModeDrafted) {
                // target rows were merged just now, the draft rows' statistics were left by the drafting calls
                const unsigned need = (1u << gb) - 1u;        // gb <= 31
                const unsigned have = GREEDY ? need : __ldcg(p.draft_ready + m_b);
                const float2* rsb = p.row_stats + (size_t)m_b * p.R;
                const int G1 = p.Gmax + 1;
                const int extra = ((have & need) == need ? 0 : BS_DEV_DRAFT_MISSING) |
                                  ((have >> 31) ? BS_DEV_NONFINITE : 0);   // a drafting pass could not sample its row
                tau = accept_finish<T, GREEDY>(p, m_b, graw, gb, al,
                                               [&](int rr) { return rr < G1 ? s_fin[rr] : __ldcg(rsb + rr); }, extra);
                if (lane == 0) p.draft_ready[m_b] = 0u;       // consumed: a later round must draft again
            } else {
                tau = accept_finish<T, GREEDY>(p, m_b, graw, gb, al, [&](int rr) { return s_fin[rr]; });
            }
            __syncwarp();
            if (lane == 0) {
                p.ticket[m_b] = 0u;                           // leave the counter clear for the next call
                if (masses) {
                    // hand the stop row over: counter first, then the word the producers look at
                    p.mass_done[m_b] = tag << 8;
                    __threadfence();                          // row statistics and counter before the word
                    *reinterpret_cast<volatile uint32_t*>(p.mass_tau + m_b) = (tag << 8) | (uint32_t)(tau + 1);
                }
            }
        }
        // ---- the CTA is done; the last one to leave clears the hand-out words and bumps the epoch ----
        if (lane == 0) {
            __threadfence();
            const unsigned gone = atomicAdd(p.sched + kSchedExit, 1u);
            if (gone == gridDim.x - 1u) {
                p.sched[kSchedCursor] = 0u;
                p.sched[kSchedMassHead] = 0u;
                p.sched[kSchedExit] = 0u;
                p.sched[kSchedEpoch] = epoch0 + 1u;
            }
        }
        return;
    }

    // ================================= consumers =================================
    Online on{-INFINITY, 0.f};
    ArgMax am{-INFINITY, INT_MAX};
    int piece_first_sg = 0;
    int pc = 0;                                               // events posted by this CTA
    int slot = 0;
    uint32_t ph = 0;
    for (;;) {
        if (!mbar_wait_warp(smem_u32(&s_full[slot]), ph)) { atomicExch(p.abort_flag, 1); return; }
        const StageMeta m = s_meta[slot];
        const int kind = m.kind & 15, flags = m.kind >> 4;
        const uint32_t sbase = smem_u32(ring + (size_t)slot * kSegBytes);
        float2 wr = make_float2(-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f);
        if (kind == kStStats) {
            const int m_sg = (m.w1 >> 19) & 0xff;
            if (flags & 1) piece_first_sg = m_sg;
            const uint32_t base = sbase + (uint32_t)tid * 16u;
            uint4 v[kVecPerThread];
            if (m.nvec == kVecPerStage) {
#pragma unroll
                for (int q = 0; q < kVecPerThread; ++q) v[q] = lds128(base + (uint32_t)(q * kConsumers) * 16u);
            } else {
#pragma unroll
                for (int q = 0; q < kVecPerThread; ++q)
                    v[q] = (q * kConsumers + tid < m.nvec) ? lds128(base + (uint32_t)(q * kConsumers) * 16u)
                                                           : neg_inf_vec<T>();
            }
            fence_reads_before_refill();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));  // the slot's data is in registers now
            if (GREEDY) argmax_add<T, kVecPerThread>(am, v, m_sg * p.seg + tid * kVec, kConsumers * kVec);
            else online_add<T, kVecPerThread>(on, v, p.c);
            if (flags & 2) {
                // ---- end of a row piece: the warp's result goes to the finisher ----
                if (GREEDY) { am = warp_best(am); wr = make_float2(am.m, __int_as_float(am.idx)); }
                else wr = warp_merge(on, p.c);
                on = Online{-INFINITY, 0.f};
                am = ArgMax{-INFINITY, INT_MAX};
            }
        } else if (kind == kStMass) {
            // 16 KB of the row pair, or 2 x 16 KB of a row sampled alone: warp w owns the w-th 1 KB piece of
            // each half and writes one mass per piece (row pair) or per half (row alone)
            MassFn f;
            f.c = p.c; f.kt = m.kt; f.kd = m.kd; f.at = m.at; f.ad = m.ad; f.bonus = (flags & 4) != 0;
            const int m_b = m.w1 & 0x1fff, m_sg = (m.w1 >> 19) & 0xff;
            const uint32_t base = sbase + (uint32_t)(warp * kRsPieceBytes + lane * 16);
            uint4 a[kRsVecPerLane], d[kRsVecPerLane];
            bool valid[kRsVecPerLane], valid2[kRsVecPerLane];
#pragma unroll
            for (int q = 0; q < kRsVecPerLane; ++q) {
                const int vi = warp * kRsPieceVecs + q * 32 + lane;
                valid[q] = vi < m.nvec;
                valid2[q] = vi < m.nvec2;
                if (valid[q]) a[q] = lds128(base + (uint32_t)(q * 512));
                if (valid2[q]) d[q] = lds128(base + (uint32_t)(kResSegBytes + q * 512));
            }
            fence_reads_before_refill();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));  // the slot's data is in registers now
            float acc = 0.f, acc2 = 0.f;
#pragma unroll
            for (int q = 0; q < kRsVecPerLane; ++q) {
                float r[kVec];
                if (valid[q]) {
                    RsElems<T>::masses(a[q], f.bonus ? a[q] : d[q], f, r);
                    float vs = 0.f;
#pragma unroll
                    for (int i = 0; i < kVec; ++i) vs += r[i];
                    acc += vs;
                }
                if (f.bonus && valid2[q]) {
                    RsElems<T>::masses(d[q], d[q], f, r);
                    float vs = 0.f;
#pragma unroll
                    for (int i = 0; i < kVec; ++i) vs += r[i];
                    acc2 += vs;
                }
            }
            acc = warp_sum(acc);
            if (f.bonus) acc2 = warp_sum(acc2);
            if (lane == 0) {
                float* out = p.resid_partial + (size_t)m_b * p.Sr + m_sg * kRsWarps + warp;
                out[0] = acc;
                if (f.bonus && m.nvec2 > 0) out[kRsWarps] = acc2;
                if (flags & 2) __threadfence();               // the chunk's masses are visible before the event
            }
        } else {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
        }
        if (++slot == nstages) { slot = 0; ph ^= 1u; }

        if (flags & 2) {
            // ---- one event for the finisher: a row piece, a mass chunk, or the end of the work ----
            const int rs = pc % kRedSlots;
            // the finisher must have taken the event that used this slot kRedSlots events ago
            if (pc >= kRedSlots &&
                !mbar_wait_warp(smem_u32(&s_redfree[rs]), (uint32_t)(pc / kRedSlots - 1) & 1u)) {
                atomicExch(p.abort_flag, 1);
                return;
            }
            if (lane == 0) {
                s_red[rs][warp] = wr;
                if (warp == 0) s_piece[rs] = PieceMeta{kind, m.w1, piece_first_sg};
                mbar_arrive(smem_u32(&s_redbar[rs]));         // release: the writes above are visible to the finisher
            }
            ++pc;
            if (kind == kStEnd) return;
        }
    }
}

static int g_stream_smem[64];          // opt-in shared memory limit per device (0 = not queried)
static bool g_attr_set[4][64];

template <typename T, bool GREEDY>
bs_status launch_verify_stream(const VerifyParams& p, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!g_stream_smem[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        g_stream_smem[dev] = v;
    }
    // two CTAs per SM: each may use half of the SM's shared memory minus the static part
    const size_t prefix_bytes = align_up(sizeof(int) * (size_t)(p.B + 1), 128);
    const size_t budget = (size_t)(g_stream_smem[dev] + 1024) / 2 - 3072;        // per CTA
    int nst = (int)((budget - prefix_bytes) / kSegBytes);
    if (nst > kMaxStages) nst = kMaxStages;
    if (nst < 2) return BS_ERR_UNSUPPORTED;
    const size_t smem = (size_t)nst * kSegBytes + prefix_bytes;
    const int variant = (Elem<T>::kDtype == BS_F32 ? 0 : 2) + (GREEDY ? 1 : 0);
    if (!g_attr_set[variant][dev]) {
        // the opt-in limit covers static + dynamic shared memory: leave room for the static part
        if (cudaFuncSetAttribute(verify_stream_kernel<T, GREEDY>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 g_stream_smem[dev] - 4096) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        g_attr_set[variant][dev] = true;
    }
    const long long items = (long long)p.B * (GREEDY ? p.Gmax + 1 : p.R) * p.nseg;       // at most: every gamma_b = Gmax
    const long long upper = (items + kChunkItems - 1) / kChunkItems;
    long long grid = 2LL * sm_count();
    if (grid > upper) grid = upper;
    if (grid < 1) grid = 1;
    return cuda_status(launch_pdl(verify_stream_kernel<T, GREEDY>, (unsigned)grid, kStreamThreads, smem, st, p, nst));
}

template bs_status launch_verify_stream<float, false>(const VerifyParams&, cudaStream_t);
template bs_status launch_verify_stream<float, true>(const VerifyParams&, cudaStream_t);
template bs_status launch_verify_stream<__nv_bfloat16, false>(const VerifyParams&, cudaStream_t);
template bs_status launch_verify_stream<__nv_bfloat16, true>(const VerifyParams&, cudaStream_t);

}  // namespace bs
