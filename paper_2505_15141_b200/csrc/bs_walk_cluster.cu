// bs_verify_walk with thread-block clusters: Algorithm 6 from its second line on, in the algorithm's own
// order -- position after position, stopping at the first rejection ("break") -- with the hand-offs between
// the CTAs that share a sequence going through distributed shared memory instead of the workspace.
//
// A sequence is shared by the nG = 2, 4 or 8 CTAs of one cluster; a cluster holds several sequences and
// interleaves them.  For position k every CTA streams its contiguous share of target row k and draft row k
// (bulk async copies into a ring of 32 KB stages, 16 consumer warps, online softmax: the pipeline of the
// row-statistics kernel).  Its finisher warp merges what its consumers produced and sends ONE message per
// position -- the (max, Z) of its part of either row -- into a mailbox of the cluster's first CTA, the
// leader of all the cluster's sequences, and arrives on the mailbox's mbarrier there.  The leader's finisher
// merges the nG messages, tests r <= min{1, P/Q} for the drafted token (the two logits at every drafted token
// were asked for when the kernel started) and writes the decision word of the sequence -- at the stop preceded
// by the constants of the residual pass -- into the shared memory of every CTA of the cluster.
//
// The producers do not wait for a decision before they stream the next position: a sequence may run up to
// `look` positions ahead of its last decided one (a mailbox per position in flight), so the decision on
// position k has to be in only before position k + look + 1 is due, and the chain "last byte reduced ->
// message -> decision -> first copy of the next position" is off the critical path.  What was streamed
// behind the stop is wasted (at most what the ring holds per CTA, since decisions are quick).  At the first
// rejection, or after the bonus row when everything passed, the producers stream the row pair of the stop
// position again (it has just been read: L2) for the residual masses; when every CTA has reported its share
// the leader runs the inverse CDF (level 2 of the resampling kernel).  In greedy mode only target rows are
// streamed, the message carries (max, arg-max), and the leader emits the arg-max of the stop row itself.
//
// A cluster waits for nobody outside itself, so the launch is an ordinary one.  Every wait is bounded; a
// wait that gives up sets the abort word and the thread leaves.  Messages of positions behind a stop may
// arrive after the leader is through with the sequence: every CTA stays until the whole cluster is done.
#include <atomic>
#include "bs_walk_common.cuh"

namespace bs {

constexpr int kClMaxSeqs = 16;                                   // sequences of one cluster (one lane of the leader each)
constexpr int kClMaxCtas = 8;
constexpr int kClLevels = 4;                                     // mailboxes per sequence: positions that may be in flight at once

struct ClMeta {                                                  // per-stage record, written by the producer
    int type, slot, b, k;
    int row;               // stats: 0 = target row k, 1 = draft row k;  mass: 1 = target row only (bonus)
    int sg, nvec, flags;   // flags bit 0: first stage of a row piece, bit 1: last stage of a piece / of the mass share,
                           // bit 2: last stage of the CTA's share of the position
    float kt, kd, at, ad;
};
struct ClEvent {                                                 // per event handed to the finisher (consumer warp 0)
    int type, slot, row, flags, k;
};
struct __align__(16) ClMail {                                    // one CTA's part of a position: target row, draft row
    float mt, zt, md, zd;                                        // greedy: (max, arg-max bits) in mt, zt
};
struct __align__(16) ClDec {                                     // what the leader's stop decision carries
    float kt, kd, at, ad;  // the constants of the residual pass
    int bonus, pad0, pad1, pad2;
};
struct __align__(16) ClPre {                                     // what the decision on one position of a sequence needs
    unsigned tw, dw;       // the 4-byte words that hold the target / draft logit at the drafted token
    float2 ds;             // drafted mode: the draft row's statistics
};

__device__ __forceinline__ uint32_t cl_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cl_id() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cl_map(const void* local, uint32_t rank) {     // the same variable in CTA `rank`
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(local)), "r"(rank));
    return ra;
}
__device__ __forceinline__ void cl_st_v4(uint32_t ra, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(ra), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void cl_st_v4u(uint32_t ra, unsigned a, unsigned b, unsigned c, unsigned d) {
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(ra), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// arrive on an mbarrier of another CTA of the cluster; what this thread wrote there before is visible to the waiter
__device__ __forceinline__ void cl_arrive(uint32_t ra) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(ra) : "memory");
}
__device__ __forceinline__ bool cl_try_wait(uint32_t bar, uint32_t parity) {       // local barrier, remote arrivals
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// The decision word of a sequence: written by the leader into every CTA after whatever the decision carries,
// polled by that CTA's producer.
__device__ __forceinline__ void cl_st_release(uint32_t ra, unsigned v) {
    asm volatile("st.release.cluster.shared::cluster.u32 [%0], %1;" ::"r"(ra), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned cl_ld_acquire(const unsigned* local) {
    unsigned v;
    asm volatile("ld.acquire.cluster.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(local)) : "memory");
    return v;
}
// Before a CTA exits: nothing written into its shared memory by another CTA of the cluster is still under way
// (messages of positions behind a stop arrive after the leader has finished with the sequence).
__device__ __forceinline__ void cl_sync_exit() {
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void cl_sync_all() {                  // every thread of every CTA of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cp_async4(void* dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(void* dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// The 4-byte word that holds element x of a row, and the element's value out of it.
template <typename T> __device__ __forceinline__ const void* word_of(const T* row, int x);
template <> __device__ __forceinline__ const void* word_of<float>(const float* row, int x) { return row + x; }
template <> __device__ __forceinline__ const void* word_of<__nv_bfloat16>(const __nv_bfloat16* row, int x) {
    return reinterpret_cast<const uint32_t*>(row) + (x >> 1);    // rows start on 16-byte boundaries
}
template <typename T> __device__ __forceinline__ float value_of(unsigned w, int x);
template <> __device__ __forceinline__ float value_of<float>(unsigned w, int) { return __uint_as_float(w); }
template <> __device__ __forceinline__ float value_of<__nv_bfloat16>(unsigned w, int x) {
    return __uint_as_float((x & 1) ? (w & 0xffff0000u) : (w << 16));
}

// The roles leave this function where their work ends; the kernel around it holds the cluster together until
// every CTA is through.
template <typename T, bool GREEDY>
__device__ __forceinline__ void walk_cluster_body(const WalkParams& p, const int nstages, const int nclusters) {
    extern __shared__ __align__(128) unsigned char dsm[];
    // layout: [nstages * 32 KB ring][tokens 16 x Gmax][uniforms 16 x Gmax][token logits 16 x Gmax]   (the last three
    // used by the leader only)
    unsigned char* ring = dsm;
    const VerifyParams& v = p.v;
    const int GP = v.Gmax > 0 ? v.Gmax : 1;
    int* s_tok = reinterpret_cast<int*>(dsm + (size_t)nstages * kSegBytes);
    float* s_u = reinterpret_cast<float*>(s_tok + kClMaxSeqs * GP);
    ClPre* s_pre = reinterpret_cast<ClPre*>(s_u + kClMaxSeqs * GP);
    __shared__ __align__(8) unsigned long long s_full[kWkStages];
    __shared__ __align__(8) unsigned long long s_empty[kWkStages];
    __shared__ __align__(8) unsigned long long s_evbar[kWkRing];
    __shared__ __align__(8) unsigned long long s_evfree[kWkRing];
    __shared__ __align__(8) unsigned long long s_mailbar[kClMaxSeqs][kClLevels];   // leader: nG messages per position
    __shared__ __align__(8) unsigned long long s_massbar[kClMaxSeqs];   // leader: nG shares of the residual masses
    __shared__ ClMail s_mail[kClMaxSeqs][kClLevels][kClMaxCtas];        // position k of a sequence uses level k % kClLevels
    __shared__ ClDec s_dec[kClMaxSeqs];                       // every CTA: what the stop decision carries
    __shared__ unsigned s_decword[kClMaxSeqs];                // every CTA: (positions decided << 1) | last one accepted
    __shared__ ClMail s_acc[kClMaxSeqs];                      // this CTA's part of the position it is streaming
    __shared__ ClMeta s_meta[kWkStages];
    __shared__ ClEvent s_ev[kWkRing];
    __shared__ float2 s_red[kWkRing][kWkWarps];
    __shared__ int s_lk[kClMaxSeqs];                          // leader: the position a sequence waits at
    __shared__ int s_lstate[kClMaxSeqs];                      // leader: 0 done, 1 waiting for messages, 2 waiting for masses
    __shared__ int s_bits[kClMaxSeqs];                        // leader: status bits found so far
    __shared__ unsigned s_ready[kClMaxSeqs];                  // leader, drafted mode: the drafted-positions word
    __shared__ int s_pstate[kClMaxSeqs];                      // producer: position and stage of every sequence

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kVec = Elem<T>::kVec;
    const int nG = p.nG;
    const uint32_t rank = cl_rank(), cid = cl_id();
    const int nslots = (int)cid < v.B ? (v.B - 1 - (int)cid) / nclusters + 1 : 0;   // sequences cid, cid + nclusters, ...

    if (tid == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), kWkWarps);
        }
        for (int s = 0; s < kWkRing; ++s) {
            mbar_init(smem_u32(&s_evbar[s]), kWkWarps);
            mbar_init(smem_u32(&s_evfree[s]), 1);
        }
        for (int s = 0; s < kClMaxSeqs; ++s) {
            for (int l = 0; l < kClLevels; ++l) mbar_init(smem_u32(&s_mailbar[s][l]), (uint32_t)nG);
            mbar_init(smem_u32(&s_massbar[s]), (uint32_t)nG);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < kClMaxSeqs) {
        s_acc[tid] = ClMail{-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f, -INFINITY, 0.f};
        s_decword[tid] = 0u;
    }
    __syncthreads();
    cl_sync_all();                                            // nobody touches a barrier of a CTA that has not set it up
    pdl_enter();                                              // gamma comes from the kernel before this one

    if (warp == kWkWarps) {
        // =============================== producer ===============================
        // Keeps the cluster's sequences moving in this CTA: streams whatever is ready and only sleeps when every
        // sequence is waiting for the leader's decision.  One lane works; the warp meets again before it leaves.
        if (lane == 0) [&]() {
        int slot = 0;
        uint32_t ph = 0;
        bool ok = true;
        auto issue = [&](const ClMeta& m, const T* src0, const T* src1, uint32_t bytes) -> bool {
            if (!mbar_wait(smem_u32(&s_empty[slot]), ph ^ 1u)) return false;
            s_meta[slot] = m;
            const uint32_t bar = smem_u32(&s_full[slot]);
            const uint32_t dst = smem_u32(ring + (size_t)slot * kSegBytes);
            if (m.type == kItemEnd) {
                mbar_arrive(bar);                              // nothing to copy: the phase completes at once
            } else {
                mbar_arrive_expect_tx(bar, src1 ? 2u * bytes : bytes);
                bulk_load(dst, src0, bytes, bar);
                if (src1) bulk_load(dst + kResSegBytes, src1, bytes, bar);
            }
            if (++slot == nstages) { slot = 0; ph ^= 1u; }
            return true;
        };
        // s_pstate[s] = the next position to stream | done << 8.  A sequence may be streamed up to p.look positions
        // past its last decided one: the decision on position k then only has to be in before position
        // k + look + 1 is due, instead of before k + 1.  What was streamed behind a stop is wasted.
        for (int s = 0; s < nslots; ++s) s_pstate[s] = 0;
        int alive = nslots;
        long long t_last = clock64();
        int rr = 0;                                            // where the next look for work ahead of a decision starts
        while (alive > 0 && ok) {
            bool progress = false;
            // First what is certainly needed -- the residual pass of a sequence that has stopped, the position after
            // an accepted one --, for every sequence; only when there is none of that, ONE position ahead of a decision.
            for (int pass = 0; pass < 2 && !progress && ok; ++pass)
            for (int q = 0; q < nslots && ok; ++q) {
                const int s = pass == 0 ? q : (rr + q) % nslots;
                if (s_pstate[s] >> 8) continue;
                const int ks = s_pstate[s];
                const int b = (int)cid + s * nclusters;
                const int g = clamp_gamma(v.gamma[b], v.Gmax);
                const unsigned w = cl_ld_acquire(&s_decword[s]);
                const int nd = (int)(w >> 1);                  // positions decided
                if (nd > 0 && !(w & 1u)) {
                    // ---- stop at k = nd - 1: this CTA's share of the residual [P_k - Q_k]_+ (rejected) or of P_k (bonus) ----
                    const int k = nd - 1;
                    if (!GREEDY) {
                        const ClDec d = s_dec[s];
                        const bool bonus = d.bonus != 0;
                        const T* tp = row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, k, v.V);
                        const T* dp = bonus ? nullptr : row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, k, v.V);
                        const int rseg = p.r.seg, rnseg = p.r.nseg;
                        const int j0 = (int)((long long)rnseg * rank / nG), j1 = (int)((long long)rnseg * (rank + 1) / nG);
                        for (int sg = j0; sg < j1 && ok; ++sg) {
                            const int e0 = sg * rseg;
                            const int n = min(rseg, v.V - e0);
                            ClMeta m;
                            m.type = kItemMass; m.slot = s; m.b = b; m.k = k; m.row = bonus ? 1 : 0; m.sg = sg;
                            m.nvec = n / kVec;
                            m.flags = (sg == j0 ? 1 : 0) | (sg == j1 - 1 ? 2 : 0);
                            m.kt = d.kt; m.kd = d.kd; m.at = d.at; m.ad = d.ad;
                            ok = issue(m, tp + e0, bonus ? nullptr : dp + e0, (uint32_t)n * (uint32_t)sizeof(T));
                        }
                    }
                    --alive;
                    s_pstate[s] = 1 << 8;
                    progress = true;
                    continue;
                }
                if (ks > g || ks > nd + (pass == 0 ? 0 : p.look)) continue;   // everything streamed / not needed yet / far enough ahead
                // ---- position ks: this CTA's share of target row ks and, below gamma, draft row ks ----
                {
                    const int k = ks;
                    const int nrows = (!GREEDY && !p.drafted && k < g) ? 2 : 1;
                    const int items = nrows * v.nseg;
                    const int i0 = (int)((long long)items * rank / nG), i1 = (int)((long long)items * (rank + 1) / nG);
                    for (int i = i0; i < i1 && ok; ++i) {
                        const int row = i / v.nseg, sg = i - row * v.nseg;
                        const T* rowp = row == 0 ? row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, k, v.V)
                                                 : row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, k, v.V);
                        const int e0 = sg * v.seg;
                        const int n = min(v.seg, v.V - e0);
                        ClMeta m;
                        m.type = kItemStats; m.slot = s; m.b = b; m.k = k; m.row = row; m.sg = sg; m.nvec = n / kVec;
                        m.flags = ((sg == 0 || i == i0) ? 1 : 0) | ((sg == v.nseg - 1 || i == i1 - 1) ? 2 : 0) |
                                  (i == i1 - 1 ? 4 : 0);
                        m.kt = m.kd = 0.f; m.at = m.ad = 1.f;
                        ok = issue(m, rowp + e0, nullptr, (uint32_t)n * (uint32_t)sizeof(T));
                    }
                    progress = true;
                    s_pstate[s] = k + 1;
                    if (pass == 1) {                           // decisions may have come in meanwhile: look again
                        rr = s + 1;
                        break;
                    }
                }
            }
            if (progress) {
                t_last = clock64();
            } else if (clock64() - t_last > kWaitCycles) {
                ok = false;
            }
        }
        if (!ok) atomicExch(v.abort_flag, 1);
        // the end marker lets the consumers and the finisher leave (also after a failed wait, if a slot frees up)
        ClMeta e;
        e.type = kItemEnd; e.slot = 0; e.b = 0; e.k = 0; e.row = 0; e.sg = 0; e.nvec = 0; e.flags = 2;
        e.kt = e.kd = 0.f; e.at = e.ad = 1.f;
        issue(e, nullptr, nullptr, 0);
        }();
        __syncwarp();
        return;
    }

    if (warp == kWkWarps + 1) {
        // =============================== finisher ===============================
        const bool leader = rank == 0;
        int remaining = leader ? nslots : 0;                  // leader: sequences not yet finished
        if (leader) {
            // ---- tokens and uniforms into shared memory; the two logits at every drafted token asked for ----
            for (int s = 0; s < nslots; ++s) {
                const int b = (int)cid + s * nclusters;
                const int graw = v.gamma[b];
                const int g = clamp_gamma(graw, v.Gmax);
                for (int j = lane; j < g; j += 32) {
                    s_tok[s * GP + j] = v.tokens[(size_t)b * v.Gmax + j];
                    if (!GREEDY) s_u[s * GP + j] = v.u_accept[(size_t)b * v.Gmax + j];
                }
                if (lane == 0) {
                    s_lk[s] = 0;
                    s_lstate[s] = 1;
                    s_bits[s] = graw != g ? BS_DEV_BAD_GAMMA : 0;
                    s_ready[s] = p.drafted ? __ldcg(v.draft_ready + b) : 0u;
                    if (p.drafted && (s_ready[s] >> 31)) s_bits[s] |= BS_DEV_NONFINITE;   // a drafting pass could not sample its row
                }
            }
            __syncwarp();
            if (!GREEDY) {
                // asynchronous 4- and 8-byte copies, waited for before the first decision: by then they have landed
                for (int i = lane; i < nslots * GP; i += 32) {
                    const int s = i / GP, j = i - s * GP;
                    const int b = (int)cid + s * nclusters;
                    const int g = clamp_gamma(v.gamma[b], v.Gmax);
                    // a field is written either here or by its copy, never by both
                    const int x = j < g ? s_tok[i] : -1;
                    if (x >= 0 && x < v.V) {
                        cp_async4(&s_pre[i].tw, word_of<T>(row_ptr(static_cast<const T*>(v.target), b, v.Gmax + 1, j, v.V), x));
                        cp_async4(&s_pre[i].dw, word_of<T>(row_ptr(static_cast<const T*>(v.draft), b, v.Gmax, j, v.V), x));
                    } else {
                        s_pre[i].tw = 0u;
                        s_pre[i].dw = 0u;
                    }
                    if (j < g && p.drafted) cp_async8(&s_pre[i].ds, v.row_stats + (size_t)b * v.R + v.Gmax + 1 + j);
                    else s_pre[i].ds = make_float2(0.f, 1.f);
                }
            }
            __syncwarp();
        }
        bool pre_landed = GREEDY;                             // leader: the copies above have been waited for

        bool ended = false;
        int ev = 0;
        long long t_idle = clock64();
        while (!ended || remaining > 0) {
            bool did = false;
            // ---- what this CTA's consumers finished ----
            if (!ended) {
                const int rs = ev % kWkRing;
                const bool there = mbar_try_wait(smem_u32(&s_evbar[rs]), (uint32_t)(ev / kWkRing) & 1u);
                if (__all_sync(0xffffffffu, there)) {
                    const ClEvent e = s_ev[rs];
                    float2 mine = make_float2(-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f);
                    if (lane < kWkWarps) mine = s_red[rs][lane];
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_evfree[rs]));   // the slot may be reused
                    ++ev;
                    did = true;
                    if (e.type == kItemEnd) {
                        ended = true;
                    } else if (e.type == kItemMass) {
                        // this CTA's share of the residual masses is written (the consumers fenced): tell the leader
                        if (lane == 0) cl_arrive(cl_map(&s_massbar[e.slot], 0));
                    } else {
                        // a piece of target row k (row 0) or of draft row k (row 1)
                        float2 out;
                        if (GREEDY) {
                            const ArgMax a = warp_best(ArgMax{mine.x, __float_as_int(mine.y)});
                            out = make_float2(a.m, __int_as_float(a.idx));
                        } else {
                            out = warp_merge(Online{mine.x, mine.y}, v.c);
                        }
                        if (lane == 0) {
                            if (e.row == 0) { s_acc[e.slot].mt = out.x; s_acc[e.slot].zt = out.y; }
                            else { s_acc[e.slot].md = out.x; s_acc[e.slot].zd = out.y; }
                            if (e.flags & 4) {
                                // the CTA's share of the position is complete: one message to the leader
                                const ClMail a = s_acc[e.slot];
                                const int lv = e.k % kClLevels;
                                cl_st_v4(cl_map(&s_mail[e.slot][lv][rank], 0), a.mt, a.zt, a.md, a.zd);
                                cl_arrive(cl_map(&s_mailbar[e.slot][lv], 0));
                                s_acc[e.slot] = ClMail{-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f, -INFINITY, 0.f};
                            }
                        }
                        __syncwarp();
                    }
                }
            }
            // ---- the leader's own work: positions whose messages are all in, sequences whose masses are all in ----
            if (leader && remaining > 0) {
                const int st = lane < nslots ? s_lstate[lane] : 0;
                bool r = false;
                if (st == 1) {
                    const int kl = s_lk[lane];
                    r = cl_try_wait(smem_u32(&s_mailbar[lane][kl % kClLevels]), (uint32_t)(kl / kClLevels) & 1u);
                }
                else if (st == 2) r = cl_try_wait(smem_u32(&s_massbar[lane]), 0u);
                unsigned todo = __ballot_sync(0xffffffffu, r);
                while (todo) {
                    const int s = __ffs(todo) - 1;
                    todo &= todo - 1;
                    did = true;
                    const int b = (int)cid + s * nclusters;
                    const int k = s_lk[s];
                    const int g = clamp_gamma(v.gamma[b], v.Gmax);
                    if (s_lstate[s] == 2) {
                        // ---- the residual masses of the stop position are complete: inverse CDF ----
                        cl_try_wait(smem_u32(&s_massbar[s]), 0u);        // every lane acquires what the CTAs released
                        __threadfence();
                        RsSeq sq;
                        sq.tau = k; sq.bonus = k >= g; sq.wgt = sq.bonus ? 1 : 2;
                        MassFn f;
                        f.c = v.c; f.bonus = sq.bonus != 0;
                        const ClDec d = s_dec[s];                        // the leader's own copy of its decision
                        f.kt = d.kt; f.kd = d.kd; f.at = d.at; f.ad = d.ad;
                        rs_level2<T>(p.r, b, sq, f);                     // token, out_tokens, out_len
                        if (lane == 0) {
                            if (p.drafted) v.draft_ready[b] = 0u;        // consumed: a later round must draft again
                            s_lstate[s] = 0;
                        }
                        __syncwarp();
                        --remaining;
                        continue;
                    }
                    // ---- position k: merge the nG messages, decide ----
                    cl_try_wait(smem_u32(&s_mailbar[s][k % kClLevels]), (uint32_t)(k / kClLevels) & 1u);   // every lane acquires the messages
                    ClMail ml{-INFINITY, GREEDY ? __int_as_float(INT_MAX) : 0.f, -INFINITY, 0.f};
                    if (lane < nG) ml = s_mail[s][k % kClLevels][lane];
                    int bits = 0;
                    bool acc = false;
                    float pj = 0.f, qj = 0.f;
                    float2 ts, ds = make_float2(0.f, 1.f);
                    const int x = k < g ? s_tok[s * GP + k] : 0;
                    const bool bad = k < g && (x < 0 || x >= v.V);
                    if (bad) bits |= BS_DEV_BAD_TOKEN;
                    if (GREEDY) {
                        ArgMax best = warp_best(ArgMax{ml.mt, __float_as_int(ml.zt)});
                        if (best.idx == INT_MAX) best.idx = 0;         // row of -inf / NaN only
                        ts = make_float2(best.m, __int_as_float(best.idx));
                        acc = k < g && !bad && x == best.idx;
                    } else {
                        const float Mt = warp_max(ml.mt);
                        const float Zt = warp_sum(ml.zt * rescale(ml.mt, Mt, v.c));
                        ts = make_float2(Mt, Zt);
                        if (!(Zt > 0.f) || !isfinite(Zt) || !isfinite(Mt)) bits |= BS_DEV_NONFINITE;
                        if (!pre_landed) {                             // the logits asked for at the start
                            cp_async_wait_all();
                            __syncwarp();
                            pre_landed = true;
                        }
                        const ClPre pre = k < g ? s_pre[s * GP + k] : ClPre{0u, 0u, make_float2(0.f, 1.f)};
                        bool missing = false;
                        if (k < g) {
                            if (p.drafted) {
                                ds = pre.ds;
                                missing = ((s_ready[s] >> k) & 1u) == 0u;
                                if (missing) bits |= BS_DEV_DRAFT_MISSING;
                            } else {
                                const float Md = warp_max(ml.md);
                                const float Zd = warp_sum(ml.zd * rescale(ml.md, Md, v.c));
                                ds = make_float2(Md, Zd);
                            }
                            if (!(ds.y > 0.f) || !isfinite(ds.y) || !isfinite(ds.x)) bits |= BS_DEV_NONFINITE;
                            if (!bad && !missing) {
                                const float tl = value_of<T>(pre.tw, x), dl = value_of<T>(pre.dw, x);
                                // log2 of the two probabilities; the ratio is formed in the log domain
                                const float lp = (tl - ts.x) * v.c - log2f(ts.y);
                                const float lq = (dl - ds.x) * v.c - log2f(ds.y);
                                pj = exp2f(lp);
                                qj = exp2f(lq);
                                // r <= min{1, P/Q}; Q(x) = 0 counts as an infinite ratio
                                acc = (lq == -INFINITY) ? true : (s_u[s * GP + k] <= fminf(1.f, exp2f(lp - lq)));
                            }
                        }
                    }
                    // ---- the decision goes to every CTA of the cluster first: they are what waits ----
                    const unsigned word = ((unsigned)(k + 1) << 1) | (acc ? 1u : 0u);
                    ClDec d;
                    d.kt = d.kd = 0.f; d.at = d.ad = 1.f; d.bonus = k >= g; d.pad0 = d.pad1 = d.pad2 = 0;
                    if (!acc && !GREEDY) {
                        MassFn::fold(ts.x, ts.y, v.c, d.kt, d.at);
                        if (k < g) MassFn::fold(ds.x, ds.y, v.c, d.kd, d.ad);
                    }
                    if (lane < nG) {
                        if (!acc && !GREEDY) {
                            const uint32_t ra = cl_map(&s_dec[s], (uint32_t)lane);
                            cl_st_v4(ra, d.kt, d.kd, d.at, d.ad);
                            cl_st_v4u(ra + 16u, (unsigned)d.bonus, 0u, 0u, 0u);
                        }
                        cl_st_release(cl_map(&s_decword[s], (uint32_t)lane), word);   // after what it carries
                    }
                    // ---- then the outputs and what the next decision will need ----
                    if (lane == 0) {
                        bits |= s_bits[s];
                        s_bits[s] = bits;
                        v.row_stats[(size_t)b * v.R + k] = ts;
                        if (!GREEDY && k < g && !p.drafted) v.row_stats[(size_t)b * v.R + v.Gmax + 1 + k] = ds;
                        if (k < g) {
                            if (v.p_tok) v.p_tok[(size_t)b * v.Gmax + k] = pj;
                            if (v.q_tok) v.q_tok[(size_t)b * v.Gmax + k] = qj;
                        }
                        if (acc) {
                            s_lk[s] = k + 1;
                        } else {
                            v.accept_len[b] = k;                     // first rejection, or k == gamma: everything passed
                            v.status[b] = bits;
                            s_lstate[s] = GREEDY ? 0 : 2;
                        }
                    }
                    if (!acc) {                                       // positions behind the stop were not looked at
                        for (int j = (k < g ? k + 1 : k) + lane; j < v.Gmax; j += 32) {
                            if (v.p_tok) v.p_tok[(size_t)b * v.Gmax + j] = 0.f;
                            if (v.q_tok) v.q_tok[(size_t)b * v.Gmax + j] = 0.f;
                        }
                        if (GREEDY) {
                            // the emitted token is the arg-max of target row k (Section 2, temperature 0)
                            int32_t* ot = p.r.out_tokens + (size_t)b * (v.Gmax + 1);
                            for (int j = lane; j <= v.Gmax; j += 32)
                                ot[j] = j < k ? s_tok[s * GP + j] : (j == k ? __float_as_int(ts.y) : -1);
                            if (lane == 0) p.r.out_len[b] = k + 1;
                            --remaining;
                        }
                    }
                    __syncwarp();
                }
            }
            if (did) {
                t_idle = clock64();
            } else if (clock64() - t_idle > kWaitCycles) {
                if (lane == 0) atomicExch(v.abort_flag, 1);
                return;
            }
        }
        return;
    }

    // ================================= consumers =================================
    Online on{-INFINITY, 0.f};
    ArgMax am{-INFINITY, INT_MAX};
    int ev = 0;                                               // events posted by this CTA
    int slot = 0;
    uint32_t ph = 0;
    for (;;) {
        if (!mbar_wait_warp(smem_u32(&s_full[slot]), ph)) { atomicExch(v.abort_flag, 1); return; }
        const ClMeta m = s_meta[slot];
        const uint32_t base = smem_u32(ring + (size_t)slot * kSegBytes);
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
        if (++slot == nstages) { slot = 0; ph ^= 1u; }

        if (m.flags & 2) {
            // ---- end of a row piece / of the mass share / of the work: one event for the finisher ----
            const int rs = ev % kWkRing;
            if (ev >= kWkRing && !mbar_wait_warp(smem_u32(&s_evfree[rs]), (uint32_t)(ev / kWkRing - 1) & 1u)) {
                atomicExch(v.abort_flag, 1);
                return;
            }
            if (lane == 0) {
                s_red[rs][warp] = wr;
                if (warp == 0) s_ev[rs] = ClEvent{m.type, m.slot, m.row, m.flags, m.k};
                mbar_arrive(smem_u32(&s_evbar[rs]));          // release: the writes above are visible to the finisher
            }
            ++ev;
            if (m.type == kItemEnd) return;
        }
    }
}

template <typename T, bool GREEDY>
__global__ void __launch_bounds__(kWkThreads, 2) verify_walk_cluster_kernel(const WalkParams p, const int nstages,
                                                                            const int nclusters) {
    walk_cluster_body<T, GREEDY>(p, nstages, nclusters);
    cl_sync_exit();
}

static std::atomic<int> g_cl_smem[64];             // opt-in shared memory limit per device (0 = not queried)
static std::atomic<int> g_cl_max[4][4][64];        // resident clusters per kernel variant and cluster size 2 / 4 / 8 (0 = not queried, -1 = none)

template <typename T, bool GREEDY>
bs_status launch_walk_cluster(WalkParams& p, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!g_cl_smem[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        g_cl_smem[dev] = v;
    }
    const int variant = (Elem<T>::kDtype == BS_F32 ? 0 : 2) + (GREEDY ? 1 : 0);
    const int GP = p.v.Gmax > 0 ? p.v.Gmax : 1;
    const size_t extra = (size_t)kClMaxSeqs * GP * (sizeof(int) + sizeof(float) + sizeof(ClPre));
    const size_t budget = (size_t)(g_cl_smem[dev] + 1024) / 2 - 13312;          // two CTAs per SM, minus the static part
    int nst = (int)((budget - extra) / kSegBytes);
    if (nst > kWkStages) nst = kWkStages;
    if (nst < 2) return BS_ERR_UNSUPPORTED;
    const size_t smem = (size_t)nst * kSegBytes + extra;
    static std::atomic<bool> attr_set[4][64];
    if (!attr_set[variant][dev]) {
        if (cudaFuncSetAttribute(verify_walk_cluster_kernel<T, GREEDY>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 g_cl_smem[dev] - 13312) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        attr_set[variant][dev] = true;
    }
    auto max_clusters = [&](int nG, cudaLaunchConfig_t& cfg) -> int {
        const int gi = nG == 8 ? 2 : (nG == 4 ? 1 : 0);
        if (!g_cl_max[variant][gi][dev]) {
            cfg.gridDim = dim3((unsigned)(nG * 16));
            int nc = 0;
            if (cudaOccupancyMaxActiveClusters(&nc, verify_walk_cluster_kernel<T, GREEDY>, &cfg) != cudaSuccess) {
                cudaGetLastError();
                nc = 0;
            }
            g_cl_max[variant][gi][dev] = nc > 0 ? nc : -1;
        }
        return g_cl_max[variant][gi][dev];
    };
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kWkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set-up overlaps the previous kernel's drain
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    // Cluster size (measured on 64 to 256 sequences of 256 KB and 608 KB rows): four CTAs per sequence unless the
    // rows are long enough to give eight CTAs four stages each per position AND the batch is small enough for
    // at most two sequences per cluster (with more, clusters of eight measured 25 to 40 % slower than clusters of
    // four); two where a row has fewer than four segments.  A cluster holds at most kClMaxSeqs sequences.
    int top = 8;
    while (top > p.v.nseg || top > p.r.nseg) top >>= 1;        // every CTA of a cluster gets a segment of every row
    int nG = 0;
    for (int c = top; c >= 2 && !nG; c >>= 1) {
        at[0].val.clusterDim.x = (unsigned)c;
        const int maxc = max_clusters(c, cfg);
        if (maxc < 1 || (p.v.B + maxc - 1) / maxc > kClMaxSeqs) continue;
        if (c == 8 && (p.v.nseg < 16 || p.v.B > 2 * maxc)) continue;
        nG = c;
    }
    if (!nG) return BS_ERR_UNSUPPORTED;
    at[0].val.clusterDim.x = (unsigned)nG;
    const int maxc = max_clusters(nG, cfg);
    const int nclusters = p.v.B < maxc ? p.v.B : maxc;
    p.nG = nG;
    // How far a sequence may run ahead of its decisions (a producer only does so when none of its sequences has
    // work that is certainly needed): all the mailboxes while a cluster has one or two sequences, one position
    // once it interleaves several (measured: +8 % / -1.5 % for the deeper run-ahead at 64 / 256 sequences).
    p.look = 2 * p.v.B <= 3 * nclusters ? kClLevels - 1 : 1;
    cfg.gridDim = dim3((unsigned)(nclusters * nG));
    return cuda_status(cudaLaunchKernelEx(&cfg, verify_walk_cluster_kernel<T, GREEDY>, p, nst, nclusters));
}

template bs_status launch_walk_cluster<float, false>(WalkParams&, cudaStream_t);
template bs_status launch_walk_cluster<float, true>(WalkParams&, cudaStream_t);
template bs_status launch_walk_cluster<__nv_bfloat16, false>(WalkParams&, cudaStream_t);
template bs_status launch_walk_cluster<__nv_bfloat16, true>(WalkParams&, cudaStream_t);

}  // namespace bs
