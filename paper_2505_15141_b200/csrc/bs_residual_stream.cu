// Pipelined resampling kernel of bs_residual_sample for rows that start on 16-byte boundaries:
// the else-branch of Algorithm 6 (one token from Norm([P - Q]_+) at the first rejected position)
// and the line after its loop (the bonus token from P), by inverse CDF in vocabulary order.
//
// A work item fills one 32 KB slot: one 16 KB segment of the row pair (target row tau_b, draft row
// tau_b) of a sequence, or two consecutive segments of the target row of a fully accepted
// sequence.  The item list is cut into gridDim.x contiguous ranges, one per CTA.
//
//   warp 16 (one lane)  producer: for each item of its range, one or two bulk async copies
//                       (TMA, no multicast) global -> shared into a ring of 2 x 16 KB slots,
//                       completion on "full" mbarriers; the per-sequence constants that fold
//                       the row statistics into the exponent travel in a per-slot record.
//   warps 0..15         consumers: warp w owns the w-th 1 KB piece of the segment, forms
//                       r_v = max(0, p_v - q_v) (or p_v) with two exps per element pair, and
//                       writes the mass of its piece; no warp ever waits for another.
//   warp 17             finisher: when the CTA's share of a sequence is done it adds the share
//                       to the sequence's arrival counter; the finisher that completes the count
//                       runs level 2 alone, while the other warps keep streaming: an fp64 scan of
//                       the piece masses picks the piece in which the cumulative mass crosses
//                       u * R, the piece (2 x 1 KB, an L2 hit) is read again, scanned in fp64 and
//                       the crossing element is the token.  The same r_v feed both levels.
//
// Every wait (mbarriers, the finisher's poll of the consumers' progress) is bounded; a wait that
// gives up sets the abort word and the thread leaves.
#include <atomic>
#include "bs_residual_level2.cuh"
#include "bs_pipeline.cuh"

namespace bs {


template <typename T>
__global__ void __launch_bounds__(kRsThreads, 2) residual_stream_kernel(const ResidParams p, const int nstages) {
    extern __shared__ __align__(128) unsigned char smem[];
    // layout: [nstages * 32 KB ring][prefix (B+1) ints]
    unsigned char* ring = smem;
    int* s_prefix = reinterpret_cast<int*>(smem + (size_t)nstages * kRsStageBytes);
    __shared__ __align__(8) unsigned long long s_full[kRsMaxStages];
    __shared__ __align__(8) unsigned long long s_empty[kRsMaxStages];
    __shared__ RsMeta s_meta[kRsMaxStages];
    __shared__ int s_scan[kRsThreads / 32];
    __shared__ unsigned int s_done;                           // consumer warps that finished a sequence share

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kVec = Elem<T>::kVec;

    if (tid == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), kRsWarps);
        }
        s_done = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    pdl_enter();                                              // accept_len and the row statistics come from the kernel before

    // ---- prefix sum of item counts over the batch (all threads, redundantly per CTA) ----
    {
        const int per = div_up(p.B, kRsThreads);
        const int b0 = tid * per;
        int local = 0;
        for (int k = 0; k < per; ++k) {
            const int b = b0 + k;
            if (b < p.B) local += rs_nitems(rs_seq(p, b), p.nseg);
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
                run += rs_nitems(rs_seq(p, b), p.nseg);
            }
        }
        if (tid == kRsThreads - 1) s_prefix[p.B] = run;
        __syncthreads();                                      // also publishes the mbarrier inits
    }
    const int total = s_prefix[p.B];
    const int lo = (int)((long long)total * blockIdx.x / gridDim.x);
    const int hi = (int)((long long)total * (blockIdx.x + 1) / gridDim.x);
    // first and last sequence that overlap [lo, hi)
    int bfirst, blast;
    {
        int l = 0, h = p.B;                                   // largest b with prefix[b] <= lo
        while (h - l > 1) {
            const int mid = (l + h) >> 1;
            if (s_prefix[mid] <= lo) l = mid; else h = mid;
        }
        bfirst = l;
        l = 0; h = p.B;                                       // largest b with prefix[b] < hi
        while (h - l > 1) {
            const int mid = (l + h) >> 1;
            if (s_prefix[mid] < hi) l = mid; else h = mid;
        }
        blast = l;
    }
    const int count = hi - lo;                                // items of this CTA: the list has unit weights
    if (count <= 0) return;

    if (warp == kRsWarps) {
        // =============================== producer ===============================
        if (lane != 0) return;
        int slot = 0;
        uint32_t ph = 0;
        for (int b = bfirst; b <= blast; ++b) {
            const RsSeq sq = rs_seq(p, b);
            int i0, i1;
            rs_items(s_prefix[b], rs_nitems(sq, p.nseg), lo, hi, i0, i1);
            if (i1 <= i0) continue;
            const float2 ts = p.row_stats[(size_t)b * p.R + rs_tslot(p, sq)];
            float kt, at, kd = 0.f, ad = 1.f;
            MassFn::fold(ts.x, ts.y, p.c, kt, at);
            const T* tp = rs_trow<T>(p, b, sq);
            const T* dp = tp;
            if (!sq.bonus) {
                const float2 ds = p.row_stats[(size_t)b * p.R + p.Gmax + 1 + sq.tau];
                MassFn::fold(ds.x, ds.y, p.c, kd, ad);
                dp = row_ptr(static_cast<const T*>(p.draft), b, p.Gmax, sq.tau, p.V);
            }
            for (int it = i0; it < i1; ++it) {
                if (!mbar_wait(smem_u32(&s_empty[slot]), ph ^ 1u)) { atomicExch(p.abort_flag, 1); return; }
                const int sg = rs_first_seg(sq, it);
                const int e0 = sg * p.seg;
                const int n = min(p.seg, p.V - e0);
                // second half of the slot: the draft row's segment, or the next segment of a row sampled alone
                const int n2 = !sq.bonus ? n : (sg + 1 < p.nseg ? min(p.seg, p.V - e0 - p.seg) : 0);
                const uint32_t bytes = (uint32_t)n * (uint32_t)sizeof(T);
                const uint32_t bytes2 = (uint32_t)n2 * (uint32_t)sizeof(T);
                RsMeta m;
                m.b = b; m.sg = sg; m.nvec = n / kVec; m.nvec2 = n2 / kVec;
                m.flags = (sq.bonus ? 1 : 0) | (it == i1 - 1 ? 2 : 0);
                m.kt = kt; m.kd = kd; m.at = at; m.ad = ad;
                s_meta[slot] = m;
                const uint32_t bar = smem_u32(&s_full[slot]);
                const uint32_t dst = smem_u32(ring + (size_t)slot * kRsStageBytes);
                mbar_arrive_expect_tx(bar, bytes + bytes2);    // releases the record to the waiters
                bulk_load(dst, tp + e0, bytes, bar);
                if (n2) bulk_load(dst + kResSegBytes, (sq.bonus ? tp + p.seg : dp) + e0, bytes2, bar);
                if (++slot == nstages) { slot = 0; ph ^= 1u; }
            }
        }
        return;
    }

    if (warp == kRsWarps + 1) {
        // =============================== finisher ===============================
        unsigned shares = 0;                                  // sequence shares of this CTA seen so far
        for (int b = bfirst; b <= blast; ++b) {
            const RsSeq sq = rs_seq(p, b);
            int i0, i1;
            rs_items(s_prefix[b], rs_nitems(sq, p.nseg), lo, hi, i0, i1);
            if (i1 <= i0) continue;
            ++shares;
            // wait until all consumer warps have written their masses of this share
            {
                const unsigned want = shares * (unsigned)kRsWarps;
                const long long t0 = clock64();
                bool ok = true;
                while (*reinterpret_cast<volatile unsigned int*>(&s_done) < want) {
                    if (clock64() - t0 > kWaitCycles) { ok = false; break; }
                    __nanosleep(64);
                }
                if (!__all_sync(0xffffffffu, ok)) {
                    if (lane == 0) atomicExch(p.abort_flag, 1);
                    return;
                }
            }
            __threadfence();
            // the ticket counts segments: an item of a row sampled alone covers two (the last one maybe one)
            const unsigned segs = sq.bonus ? (unsigned)(min(2 * i1, p.nseg) - 2 * i0) : (unsigned)(i1 - i0);
            unsigned old = 0;
            if (lane == 0) old = atomicAdd(p.ticket + b, segs);
            old = __shfl_sync(0xffffffffu, old, 0);
            if (old + segs == (unsigned)p.nseg) {
                __threadfence();
                MassFn f;
                f.c = p.c;
                f.bonus = sq.bonus;
                const float2 ts = p.row_stats[(size_t)b * p.R + rs_tslot(p, sq)];
                MassFn::fold(ts.x, ts.y, p.c, f.kt, f.at);
                f.kd = 0.f; f.ad = 1.f;
                if (!sq.bonus) {
                    const float2 ds = p.row_stats[(size_t)b * p.R + p.Gmax + 1 + sq.tau];
                    MassFn::fold(ds.x, ds.y, p.c, f.kd, f.ad);
                }
                rs_level2<T>(p, b, sq, f);
            }
        }
        return;
    }

    // ================================= consumers =================================
    int slot = 0;
    uint32_t ph = 0;
    for (int k = 0; k < count; ++k) {
        if (!mbar_wait_warp(smem_u32(&s_full[slot]), ph)) { atomicExch(p.abort_flag, 1); return; }
        const RsMeta m = s_meta[slot];
        MassFn f;
        f.c = p.c; f.kt = m.kt; f.kd = m.kd; f.at = m.at; f.ad = m.ad; f.bonus = (m.flags & 1) != 0;
        const uint32_t base = smem_u32(ring + (size_t)slot * kRsStageBytes) + (uint32_t)(warp * kRsPieceBytes + lane * 16);
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
        // row pair: one mass per piece from both halves; row alone: one mass per half
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
            float* out = p.resid_partial + (size_t)m.b * p.S + m.sg * kRsWarps + warp;
            out[0] = acc;
            if (f.bonus && m.nvec2 > 0) out[kRsWarps] = acc2;
            if (m.flags & 2) {                                // this CTA's share of the sequence ends here
                __threadfence();
                atomicAdd(&s_done, 1u);
            }
        }
        if (++slot == nstages) { slot = 0; ph ^= 1u; }
    }
}

static std::atomic<int> g_rs_smem[64];          // opt-in shared memory limit per device (0 = not queried)
static std::atomic<bool> g_rs_attr[2][64];

template <typename T>
bs_status launch_residual_stream(const ResidParams& p, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (!g_rs_smem[dev]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        g_rs_smem[dev] = v;
    }
    // two CTAs per SM: each may use half of the SM's shared memory minus the static part
    const size_t prefix_bytes = align_up(sizeof(int) * (size_t)(p.B + 1), 128);
    const size_t budget = (size_t)(g_rs_smem[dev] + 1024) / 2 - 3072;
    int nst = (int)((budget - prefix_bytes) / kRsStageBytes);
    if (nst > kRsMaxStages) nst = kRsMaxStages;
    if (nst < 2) return BS_ERR_UNSUPPORTED;
    const size_t smem = (size_t)nst * kRsStageBytes + prefix_bytes;
    const int variant = Elem<T>::kDtype == BS_F32 ? 0 : 1;
    if (!g_rs_attr[variant][dev]) {
        if (cudaFuncSetAttribute(residual_stream_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 g_rs_smem[dev] - 4096) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        g_rs_attr[variant][dev] = true;
    }
    long long grid = 2LL * sm_count();
    const long long items = (long long)p.B * p.nseg;
    if (grid > items) grid = items;
    if (grid < 1) grid = 1;
    return cuda_status(launch_pdl(residual_stream_kernel<T>, (unsigned)grid, kRsThreads, smem, st, p, nst));
}

template bs_status launch_residual_stream<float>(const ResidParams&, cudaStream_t);
template bs_status launch_residual_stream<__nv_bfloat16>(const ResidParams&, cudaStream_t);

}  // namespace bs
