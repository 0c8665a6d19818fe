// Pipelined row-statistics kernel of bs_softmax_verify for rows that start on 16-byte
// boundaries (V * sizeof(element) a multiple of 16): softmax with temperature (Section 2 of the
// paper) and the accept loop of Algorithm 6.
//
// The flat list of work items (one item = one 32 KB segment of one valid row; ragged gamma_b
// handled through a prefix sum over the batch) is cut into gridDim.x contiguous ranges, one
// per CTA, so every CTA streams the same number of bytes (+-1 segment) and mostly whole rows.
//
//   warp 16 (one lane) producer: walks its range, and for each segment arms a "full" mbarrier
//                      with the byte count and issues one bulk async copy (TMA, no multicast)
//                      global -> shared into a ring of 32 KB slots.
//   warps 0..15        consumers: wait for the slot, read it with conflict-free 128-bit shared
//                      loads, update a per-thread online softmax state (chunk max first, then
//                      ONE exp per logit), release the slot through an "empty" mbarrier.
//
//   warp 17            finisher: takes the row pieces the consumers finish (a small ring of
//                      per-warp results in shared memory), merges them, publishes the piece and
//                      does what the piece completes, so the consumers never leave the stream.
//
// The per-thread state lives across all segments of a row piece; it is reduced only when the
// row (or the CTA's range) ends.  Every piece is published as a partial and counted on one atomic
// ticket per sequence; the finisher whose piece completes the count merges all rows of the
// sequence (one lane per row) and runs the accept scan.  Nobody waits on another CTA.  All waits
// on mbarriers are bounded; a wait that gives up sets the abort word and the thread leaves.
#include <atomic>
#include "bs_verify_common.cuh"
#include "bs_pipeline.cuh"

namespace bs {

constexpr int kConsumerWarps = 16;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kStreamThreads = kConsumers + 64;                   // + producer warp + finisher warp
constexpr int kVecPerStage = kSegBytes / 16;                     // 2048
constexpr int kVecPerThread = kVecPerStage / kConsumers;         // 4
constexpr int kMaxStages = 3;
constexpr int kRedSlots = 8;                                     // row-piece results the consumers may run ahead of the finisher
static_assert(kVecPerThread * kConsumers == kVecPerStage, "stage must divide evenly over the consumers");

// Per-stage record written by the producer: w0 = nvec | flags << 16, w1 = b | lr << 13 | sg << 19
// (b < 2^13, lr < 2^6, sg < 2^8).  flags bit 0: first stage of a row piece, bit 1: last stage.
struct StageMeta {
    int w0, w1;
};
// Per finished row piece, written by consumer warp 0: w1 of the piece's last stage; first segment
// of the piece in the low half, bit 16 set on the CTA's last piece.
struct PieceMeta {
    int w1, first_sg;
};
static_assert(BS_MAX_BATCH <= (1 << 13) && 2 * BS_MAX_GAMMA + 1 < (1 << 6) &&
              BS_MAX_VOCAB / (kSegBytes / 4) <= (1 << 8), "StageMeta packing");

template <typename T, bool GREEDY>
__global__ void __launch_bounds__(kStreamThreads, 2) verify_stream_kernel(const VerifyParams p, const int nstages) {
    extern __shared__ __align__(128) unsigned char smem[];
    // layout: [nstages * 32 KB ring][prefix (B+1) ints]
    unsigned char* ring = smem;
    int* s_prefix = reinterpret_cast<int*>(smem + (size_t)nstages * kSegBytes);
    __shared__ __align__(8) unsigned long long s_full[kMaxStages];
    __shared__ __align__(8) unsigned long long s_empty[kMaxStages];
    // one reduction barrier per s_red slot: a warp may run several row pieces ahead of another,
    // so arrivals of different pieces must never meet on one barrier
    __shared__ __align__(8) unsigned long long s_redbar[kRedSlots];
    __shared__ __align__(8) unsigned long long s_redfree[kRedSlots];
    __shared__ PieceMeta s_piece[kRedSlots];
    __shared__ float2 s_fin[2 * BS_MAX_GAMMA + 1];            // merged row statistics of the sequence being finished
    __shared__ __align__(8) StageMeta s_meta[kMaxStages];
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
    const int lo = (int)((long long)total * blockIdx.x / gridDim.x);
    const int hi = (int)((long long)total * (blockIdx.x + 1) / gridDim.x);
    const int count = hi - lo;
    if (count <= 0) return;

    if (warp == kConsumerWarps) {
        // =============================== producer ===============================
        if (lane != 0) return;
        // first item of the range -> (sequence, local row, segment)
        int b, lr, sg, g, rows_b;
        {
            int l = 0, h = p.B;                               // largest b with prefix[b] <= lo
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
        int slot = 0;
        uint32_t ph = 0;
        for (int k = 0; k < count; ++k) {
            if (!mbar_wait(smem_u32(&s_empty[slot]), ph ^ 1u)) { atomicExch(p.abort_flag, 1); return; }
            const T* rowp = mode_row<T>(p, b, lr, g);
            const int e0 = sg * p.seg;
            const int n = min(p.seg, p.V - e0);
            const uint32_t bytes = (uint32_t)n * (uint32_t)sizeof(T);
            const int flags = ((sg == 0 || k == 0) ? 1 : 0) | ((sg == p.nseg - 1 || k == count - 1) ? 2 : 0);
            StageMeta m;
            m.w0 = (n / kVec) | (flags << 16);
            m.w1 = b | (lr << 13) | (sg << 19);
            s_meta[slot] = m;
            const uint32_t bar = smem_u32(&s_full[slot]);
            mbar_arrive_expect_tx(bar, bytes);                // releases the meta write to the waiters
            bulk_load(smem_u32(ring + (size_t)slot * kSegBytes), rowp + e0, bytes, bar);
            // advance to the next item
            if (++sg == p.nseg) {
                sg = 0;
                if (++lr == rows_b) {
                    lr = 0;
                    do {                                      // next sequence that contributes rows
                        ++b;
                        if (b < p.B) {
                            g = clamp_gamma(p.gamma[b], p.Gmax);
                            rows_b = mode_rows<GREEDY>(p, g);
                        }
                    } while (b < p.B && rows_b == 0);
                }
            }
            if (++slot == nstages) { slot = 0; ph ^= 1u; }
        }
        return;
    }

    if (warp == kConsumerWarps + 1) {
        // =============================== finisher ===============================
        // Takes the row pieces the consumers finish, in order: merges the 16 warp results,
        // publishes the piece, and does whatever the piece completes (row merge, accept scan).
        // The consumers never wait for any of this.
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
            float2 out;
            if (GREEDY) {
                ArgMax a = warp_best(ArgMax{mine.x, __float_as_int(mine.y)});
                out = make_float2(a.m, __int_as_float(a.idx));
            } else {
                out = warp_merge(Online{mine.x, mine.y}, p.c);
            }
            // ---- publish the piece; the finisher that completes the sequence does the rest ----
            const int m_b = pm.w1 & 0x1fff, m_lr = (pm.w1 >> 13) & 0x3f, m_sg = (pm.w1 >> 19) & 0xff;
            const int first_sg = pm.first_sg & 0xffff;
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
            if (old + (unsigned)piece_len == (unsigned)(rows_mb * p.nseg)) {
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
                if (p.mode == kModeDraft) {
                    // the draft row's statistics are in place; greedy drafting ends here
                    if (lane == 0) {
                        if (GREEDY) p.draft_out[(size_t)m_b * p.Gmax + p.position] = __float_as_int(s_fin[r].y);
                        __threadfence();
                        atomicOr(p.draft_ready + m_b, 1u << p.position);
                    }
                } else if (p.mode == kModeDrafted) {
                    // target rows were merged just now, the draft rows' statistics were left by the drafting calls
                    const unsigned need = (1u << gb) - 1u;        // gamma <= 31
                    const unsigned have = GREEDY ? need : __ldcg(p.draft_ready + m_b);
                    const float2* rsb = p.row_stats + (size_t)m_b * p.R;
                    const int G1 = p.Gmax + 1;
                    accept_finish<T, GREEDY>(p, m_b, graw, gb, al,
                                             [&](int rr) { return rr < G1 ? s_fin[rr] : __ldcg(rsb + rr); },
                                             ((have & need) == need ? 0 : BS_DEV_DRAFT_MISSING) |
                                                 ((have >> 31) ? BS_DEV_NONFINITE : 0));   // a drafting pass could not sample its row
                    if (lane == 0) p.draft_ready[m_b] = 0u;       // consumed: a later round must draft again
                } else {
                    accept_finish<T, GREEDY>(p, m_b, graw, gb, al, [&](int rr) { return s_fin[rr]; });
                }
                if (lane == 0) p.ticket[m_b] = 0u;                // leave the counter clear for the next call
            }
            if (pm.first_sg >> 16) break;                     // that was the CTA's last piece
        }
        return;
    }

    // ================================= consumers =================================
    Online on{-INFINITY, 0.f};
    ArgMax am{-INFINITY, INT_MAX};
    int piece_first_sg = 0;
    int pc = 0;                                               // row pieces finished by this CTA
    int slot = 0;
    uint32_t ph = 0;
    for (int k = 0; k < count; ++k) {
        if (!mbar_wait_warp(smem_u32(&s_full[slot]), ph)) { atomicExch(p.abort_flag, 1); return; }
        const StageMeta m = s_meta[slot];
        const int nvec = m.w0 & 0xffff, flags = m.w0 >> 16;
        const int m_sg = (m.w1 >> 19) & 0xff;
        if (flags & 1) piece_first_sg = m_sg;
        const uint32_t base = smem_u32(ring + (size_t)slot * kSegBytes) + (uint32_t)tid * 16u;
        uint4 v[kVecPerThread];
        if (nvec == kVecPerStage) {
#pragma unroll
            for (int q = 0; q < kVecPerThread; ++q) v[q] = lds128(base + (uint32_t)(q * kConsumers) * 16u);
        } else {
#pragma unroll
            for (int q = 0; q < kVecPerThread; ++q)
                v[q] = (q * kConsumers + tid < nvec) ? lds128(base + (uint32_t)(q * kConsumers) * 16u) : neg_inf_vec<T>();
        }
        fence_reads_before_refill();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));  // the slot's data is in registers now
        if (GREEDY) argmax_add<T, kVecPerThread>(am, v, m_sg * p.seg + tid * kVec, kConsumers * kVec);
        else online_add<T, kVecPerThread>(on, v, p.c);
        if (++slot == nstages) { slot = 0; ph ^= 1u; }

        if (flags & 2) {
            // ---- end of a row piece: hand the warp's result to the finisher ----
            float2 wr;
            if (GREEDY) { am = warp_best(am); wr = make_float2(am.m, __int_as_float(am.idx)); }
            else wr = warp_merge(on, p.c);
            const int rs = pc % kRedSlots;
            // the finisher must have taken the piece that used this slot kRedSlots pieces ago
            if (pc >= kRedSlots &&
                !mbar_wait_warp(smem_u32(&s_redfree[rs]), (uint32_t)(pc / kRedSlots - 1) & 1u)) {
                atomicExch(p.abort_flag, 1);
                return;
            }
            if (lane == 0) {
                s_red[rs][warp] = wr;
                if (warp == 0) s_piece[rs] = PieceMeta{m.w1, piece_first_sg | ((k == count - 1) ? (1 << 16) : 0)};
                mbar_arrive(smem_u32(&s_redbar[rs]));         // release: the writes above are visible to the finisher
            }
            on = Online{-INFINITY, 0.f};
            am = ArgMax{-INFINITY, INT_MAX};
            ++pc;
        }
    }
}

static std::atomic<int> g_stream_smem[64];          // opt-in shared memory limit per device (0 = not queried)
static std::atomic<bool> g_attr_set[4][64];

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
    const long long upper = (long long)p.B * (GREEDY ? p.Gmax + 1 : p.R) * p.nseg;
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
