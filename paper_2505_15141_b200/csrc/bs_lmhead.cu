// bs_lmhead_verify: the last step of the parallel target / draft evaluation of Algorithm 6
// (second line) fused with the verification statistics -- logits = H W on the tensor cores,
// softmax statistics (Section 2) in the epilogue, then the accept loop of Algorithm 6.
//
//   H  [M, d]  bf16, d contiguous   (M = B * (Gmax + 1) target rows, B * Gmax draft rows)
//   W  [d, V]  bf16, V contiguous   (the output embedding, streamed once from HBM)
//   out[M, V]  fp32                 (kept for the resampling step)
//
// One persistent CTA per SM walks a static list of 128 x BN or 256 x BN output tiles (target product first,
// then the draft product; tiles that share a slice of W are adjacent in the list so the slice
// comes from L2 the second time).  Per CTA:
//   warp 0 (one lane)   TMA producer: per 64-deep k-block one 128 x 64 box of H (K-major,
//                       128-byte swizzle, rows past M zero-filled by the tensor map) and BN / 64
//                       boxes of 64 (k) x 64 (n) of W (N-major, 128-byte swizzle) into a ring of
//                       shared-memory stages, completion on "full" mbarriers.
//   warp 1 (one lane)   issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32, M = 128, N = BN,
//                       K = 16) on shared-memory descriptors, accumulating in tensor memory;
//                       tcgen05.commit releases the stage ("empty") and, after the last
//                       k-block, publishes the accumulator ("tmem_full").
//   warps 2..9          epilogue: tcgen05.ld their 32 lanes of the accumulator, 32 columns at a
//                       time (four lane quarters x two column halves); every thread owns one
//                       output row, so the running (max, sum exp) or (max, arg-max) of that row
//                       over its half tile needs no shuffle; the fp32 logits leave through a 4 KB
//                       staging block per warp and a TMA store of 32 rows x 32 columns (whole
//                       128-byte lines; a thread storing its own row would touch 32 lines per
//                       instruction), the per-(row, half tile) statistics go to a partial buffer.
// A second small kernel merges the partials of every row, stores the row statistics in the
// workspace (where bs_residual_sample reads them) and runs the accept scan.
//
// Every mbarrier wait is bounded (about a second); a wait that gives up sets the abort word,
// every role leaves its loop, the CTA meets at the final barrier and tensor memory is freed.
#include <atomic>
#include "bs_verify_common.cuh"
#include "bs_pipeline.cuh"

#include <cuda.h>          // CUtensorMap and its enums; the encoder is looked up at run time

namespace bs {

constexpr int kLmBM = 128;                 // tile rows = UMMA M = tensor-memory lanes
constexpr int kLmBK = 64;                  // k-extent of a stage: 64 bf16 = one 128-byte swizzle row
constexpr int kLmUK = 16;                  // k-extent of one tcgen05.mma for 16-bit operands
constexpr int kLmEpiWarps = 8;             // epilogue warps: 4 lane quarters x 2 column halves
constexpr int kLmThreads = 64 + 32 * kLmEpiWarps;   // producer warp, MMA warp, epilogue warps
constexpr int kLmABytes = kLmBM * kLmBK * 2;                      // 16 KB of H per stage
constexpr int kLmChunkBytes = kLmBK * 128;                        // 64 k-rows x 64 n (128 B) of W = 8 KB
constexpr int kLmTmemCols = 512;           // two fp32 accumulators of up to 256 columns
constexpr int kLmOutBoxBytes = 32 * 32 * 4;                       // staging block of one epilogue warp
constexpr int kLmOutBytes = kLmEpiWarps * kLmOutBoxBytes;         // 32 KB behind the stages

struct LmProduct {
    float* out;            // [M, V] fp32 logits
    int M;                 // rows of H
    int KB;                // k-blocks: ceil(d / 64)
    int MT;                // row tiles of one CTA: ceil(M / (128 * MH))
    int rows_per_seq;      // Gmax + 1 (target) or Gmax (draft)
    int slot0;             // row slot of a sequence's first row in the statistics: 0 or Gmax + 1
};

struct LmParams {
    LmProduct prod[2];
    int nprod;             // 2, or 1 when there are no draft rows (greedy mode, Gmax = 0)
    int V, NT, R;          // vocabulary, column tiles ceil(V / BN), row slots per sequence 2 Gmax + 1
    float c;               // log2(e) / temperature
    float2* partial;       // [B * R, 2 NT] statistics per row and half column tile
    int32_t* abort_flag;
};

// ---- PTX wrappers ---------------------------------------------------------------------------

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}
// shared -> global store of one box; completion is tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(tm), "r"(x), "r"(y), "r"(src) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() {        // the stores issued so far have read their source
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_all() {         // ... and have been written
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {       // arrives on `bar` when all earlier MMAs are done
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], one 128 x N x 16 step
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory: thread = lane, v[i] = column i
__device__ __forceinline__ void tc_load_32cols(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor (tcgen05): start address, leading / stride byte offsets in
// 16-byte units, descriptor version 1 (bits 46-47), 128-byte swizzle (value 2 in bits 61-63).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor of kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9 and
// 10-12 = 1), A K-major (bit 15 = 0), B N-major (bit 16 = 1), N / 8 in bits 17-22, M / 16 in bits 24-28.
__host__ __device__ constexpr uint32_t lm_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kLmBM >> 4) << 24);
}

struct LmTile {
    int prod, nt, mt;
};
__device__ __forceinline__ LmTile lm_tile(const LmParams& p, int t) {
    const int t0 = p.prod[0].MT * p.NT;
    LmTile r;
    r.prod = t >= t0 ? 1 : 0;
    if (r.prod) t -= t0;
    const int mtn = p.prod[r.prod].MT;
    r.nt = t / mtn;
    r.mt = t - r.nt * mtn;
    return r;
}

// MH = row tiles of 128 that one CTA multiplies against the same 64 x BN block of W per stage.
//   MH = 1  (M <= 128): two accumulators of BN columns alternate between tiles, so the epilogue
//           of a tile runs under the k-loop of the next; 4 stages of 16 + 32 KB.
//   MH = 2  (larger M): a 256 x BN tile, both accumulators belong to the current tile; every byte
//           of W brought into shared memory feeds twice the MMAs (half the L2 -> SM traffic per
//           flop, twice the time a stage lasts); 3 stages of 32 + 32 KB.
template <int BN, int MH, int STAGES, bool GREEDY>
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_gemm_kernel(const __grid_constant__ CUtensorMap tm_h0, const __grid_constant__ CUtensorMap tm_w0,
                   const __grid_constant__ CUtensorMap tm_h1, const __grid_constant__ CUtensorMap tm_w1,
                   const __grid_constant__ CUtensorMap tm_o0, const __grid_constant__ CUtensorMap tm_o1,
                   const LmParams p) {
    constexpr int kChunks = BN / 64;
    constexpr int kBBytes = kChunks * kLmChunkBytes;
    constexpr int kStageBytes = MH * kLmABytes + kBBytes;
    constexpr int kHalfCols = BN / 2;                         // columns one epilogue warp covers
    static_assert(BN % 64 == 0 && BN >= 64 && 2 * BN <= kLmTmemCols, "tile width");
    static_assert(MH == 1 || MH == 2, "row tiles per CTA");
    static_assert(kStageBytes % 1024 == 0, "stages must keep the 1024-byte swizzle alignment");

    extern __shared__ unsigned char lm_smem_raw[];
    // the swizzle pattern is a function of the address bits: stage bases must be 1024-byte aligned
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(lm_smem_raw) + 1023) &
                                                           ~(uintptr_t)1023);
    unsigned char* out_stage = smem + (size_t)STAGES * kStageBytes;   // 1024-byte aligned like the stages
    __shared__ __align__(8) unsigned long long s_full[STAGES];
    __shared__ __align__(8) unsigned long long s_empty[STAGES];
    __shared__ __align__(8) unsigned long long s_tmem_full[2];
    __shared__ __align__(8) unsigned long long s_tmem_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int total_tiles = p.prod[0].MT * p.NT + (p.nprod > 1 ? p.prod[1].MT * p.NT : 0);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&s_full[s]), 1);
            mbar_init(smem_u32(&s_empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&s_tmem_full[a]), 1);
            mbar_init(smem_u32(&s_tmem_empty[a]), kLmEpiWarps);   // one arrival per epilogue warp
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                          // tensor memory: whole warp allocates
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"(kLmTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    pdl_wait();                                               // H may come from the kernel before this one

    // Accumulator used by tile number `it` of this CTA for row half `h`.  The MMA issuer and the
    // epilogue warps each count how often an accumulator has been used (`uses`): the parity of
    // that count is the phase of its two barriers.
    auto acc_of = [](int it, int h) { return MH == 1 ? (it & 1) : h; };

    if (warp == 0) {
        // ================================ TMA producer ================================
        if (lane == 0) {
            // W is read by one CTA per column tile (evict first) or by several at about the same
            // time (normal priority, so that the later ones find it in L2); H is re-read by every
            // column tile.
            const bool w_once = p.prod[0].MT == 1 && (p.nprod == 1 || p.prod[1].MT == 1);
            const uint64_t pol_w = w_once ? policy_evict_first() : policy_evict_normal();
            const uint64_t pol_h = policy_evict_last();
            int slot = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const LmTile tl = lm_tile(p, t);
                const CUtensorMap* th = tl.prod ? &tm_h1 : &tm_h0;
                const CUtensorMap* tw = tl.prod ? &tm_w1 : &tm_w0;
                const int KB = p.prod[tl.prod].KB;
                const int n0 = tl.nt * BN;
                const int m0 = tl.mt * (kLmBM * MH);
                const int halves = (MH == 2 && m0 + kLmBM < p.prod[tl.prod].M) ? 2 : 1;
                const int chunks = min(kChunks, (p.V - n0 + 63) / 64);      // chunks that hold any column < V
                const uint32_t tx = (uint32_t)(halves * kLmABytes + chunks * kLmChunkBytes);
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(smem_u32(&s_empty[slot]), ph ^ 1u) || s_abort) { ok = false; break; }
                    const uint32_t bar = smem_u32(&s_full[slot]);
                    const uint32_t sa = smem_u32(smem + (size_t)slot * kStageBytes);
                    mbar_arrive_expect_tx(bar, tx);
                    for (int h = 0; h < halves; ++h)
                        tma_load_2d(sa + h * kLmABytes, th, kb * kLmBK, m0 + h * kLmBM, bar, pol_h);
                    for (int j = 0; j < chunks; ++j)
                        tma_load_2d(sa + MH * kLmABytes + j * kLmChunkBytes, tw, n0 + j * 64, kb * kLmBK, bar, pol_w);
                    if (++slot == STAGES) { slot = 0; ph ^= 1u; }
                }
            }
            if (!ok) { s_abort = 1; atomicExch(p.abort_flag, 1); }
        }
    } else if (warp == 1) {
        // ================================= MMA issuer =================================
        if (lane == 0) {
            constexpr uint32_t idesc = lm_idesc(BN);
            int slot = 0;
            uint32_t ph = 0;
            uint32_t uses[2] = {0u, 0u};
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                const LmTile tl = lm_tile(p, t);
                const int KB = p.prod[tl.prod].KB;
                const int m0 = tl.mt * (kLmBM * MH);
                const int halves = (MH == 2 && m0 + kLmBM < p.prod[tl.prod].M) ? 2 : 1;
                for (int kb = 0; kb < KB && ok; ++kb) {
                    if (!mbar_wait(smem_u32(&s_full[slot]), ph) || s_abort) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)slot * kStageBytes);
                    const uint32_t sb = sa + MH * kLmABytes;
                    for (int h = 0; h < halves; ++h) {
                        const int acc = acc_of(it, h);
                        if (kb == 0) {
                            // the epilogue must have drained this accumulator (its previous use)
                            if (!mbar_wait(smem_u32(&s_tmem_empty[acc]), (uses[acc] & 1u) ^ 1u) || s_abort) { ok = false; break; }
                            tc_fence_after();
                        }
                        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
#pragma unroll
                        for (int k = 0; k < kLmBK / kLmUK; ++k) {
                            // A, K-major: rows of 128 B, 8-row groups 1024 B apart; a k-step is 32 B inside the row
                            const uint64_t a_desc = smem_desc(sa + h * kLmABytes + k * (kLmUK * 2), 16, 1024);
                            // B, N-major: 64-column chunks kLmChunkBytes apart (leading), 8-k-row groups
                            // 1024 B apart (stride); a k-step is 16 rows of 128 B
                            const uint64_t b_desc = smem_desc(sb + k * (kLmUK * 128), kLmChunkBytes, 1024);
                            tc_mma_bf16(d_tmem, a_desc, b_desc, idesc, (kb | k) ? 1u : 0u);
                        }
                    }
                    if (!ok) break;
                    tc_commit(smem_u32(&s_empty[slot]));       // the stage may be refilled once these MMAs retire
                    if (++slot == STAGES) { slot = 0; ph ^= 1u; }
                }
                if (ok)
                    for (int h = 0; h < halves; ++h) {
                        tc_commit(smem_u32(&s_tmem_full[acc_of(it, h)]));
                        ++uses[acc_of(it, h)];
                    }
            }
            if (!ok) { s_abort = 1; atomicExch(p.abort_flag, 1); }
        }
    } else {
        // ================================== epilogue ==================================
        // warps 2..9: lane quarter warp % 4 of the accumulator (the lanes a warp may read), column
        // half (warp - 2) / 4 of the tile
        const int quarter = warp & 3;
        const int chalf = (warp - 2) >> 2;
        uint32_t uses[2] = {0u, 0u};
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
            const LmTile tl = lm_tile(p, t);
            const LmProduct& pr = p.prod[tl.prod];
            const int m0 = tl.mt * (kLmBM * MH);
            const int halves = (MH == 2 && m0 + kLmBM < pr.M) ? 2 : 1;
            for (int h = 0; h < halves && ok; ++h) {
                const int acc = acc_of(it, h);
                // warp-uniform outcome: the tensor-memory loads below need the whole warp
                const bool arrived = mbar_wait_warp(smem_u32(&s_tmem_full[acc]), uses[acc] & 1u);
                ++uses[acc];
                const int aborted = __shfl_sync(0xffffffffu, (int)s_abort, 0);
                if (!arrived || aborted) { ok = false; break; }
                tc_fence_after();
                const int row = m0 + h * kLmBM + quarter * 32 + lane;
                const bool row_ok = row < pr.M;
                const int n0 = tl.nt * BN + chalf * kHalfCols;
                const int ncols = max(0, min(kHalfCols, p.V - n0));
                const int row0 = m0 + h * kLmBM + quarter * 32;
                const uint32_t obuf = smem_u32(out_stage + (size_t)(warp - 2) * kLmOutBoxBytes);
                Online on{-INFINITY, 0.f};
                ArgMax am{-INFINITY, INT_MAX};
                if (m0 + h * kLmBM + quarter * 32 < pr.M) {   // some row of this warp exists
                    for (int c0 = 0; c0 < ncols; c0 += 32) {
                        uint32_t v[32];
                        tc_load_32cols(tmem_base + ((uint32_t)(quarter * 32) << 16) +
                                           (uint32_t)(acc * BN + chalf * kHalfCols + c0), v);
                        const int nv = min(32, ncols - c0);   // valid columns of this group (a multiple of 4)
                        if (row_ok) {
                            if (GREEDY) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) {
                                    const float x = __uint_as_float(v[i]);
                                    if (i < nv && x > am.m) { am.m = x; am.idx = n0 + c0 + i; }
                                }
                            } else {
                                float cm = -INFINITY;
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (i < nv) cm = fmaxf(cm, __uint_as_float(v[i]));
                                on.raise_to(cm, p.c);
                                if (on.m > -INFINITY) {
                                    const float nm = -on.m * p.c;
                                    float a0 = 0.f, a1 = 0.f;
#pragma unroll
                                    for (int i = 0; i < 32; i += 2) {
                                        if (i < nv) {
                                            a0 += ex2(fmaf(__uint_as_float(v[i]), p.c, nm));
                                            a1 += ex2(fmaf(__uint_as_float(v[i + 1]), p.c, nm));
                                        }
                                    }
                                    const float dl = fmaf(on.m, p.c, nm);      // rounding error of nm, undone to first order
                                    on.s = fmaf(a0 + a1, fmaf(-dl, 0.69314718f, 1.f), on.s);
                                }
                            }
                        }
                        // The 32 x 32 block leaves through shared memory: row = lane, 16-byte chunk j of a
                        // row sits at j ^ (row % 8) (the 128-byte swizzle the tensor map undoes), so the
                        // eight lanes of a quarter warp hit eight different chunks.  Rows past M and
                        // columns past V are clipped by the tensor map.
                        if (lane == 0) tma_store_wait_read();     // the block before this one has been read
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            sts128(obuf + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4)), v[4 * j], v[4 * j + 1],
                                   v[4 * j + 2], v[4 * j + 3]);
                        fence_writes_before_bulk_store();
                        __syncwarp();
                        if (lane == 0) tma_store_2d(tl.prod ? &tm_o1 : &tm_o0, obuf, n0 + c0, row0);
                    }
                }
                // accumulator drained: hand it back before the bookkeeping
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_tmem_empty[acc]));
                if (row_ok) {
                    const int b = row / pr.rows_per_seq;
                    const int j = row - b * pr.rows_per_seq;
                    p.partial[((size_t)b * p.R + pr.slot0 + j) * (2 * p.NT) + 2 * tl.nt + chalf] =
                        GREEDY ? make_float2(am.m, __int_as_float(am.idx)) : make_float2(on.m, on.s);
                }
            }
        }
        if (lane == 0) tma_store_wait_all();                  // shared memory is given up only after the last store
        if (!ok && lane == 0) { s_abort = 1; atomicExch(p.abort_flag, 1); }
    }

    // ---- all roles meet; tensor memory goes back ----
    pdl_release();                                            // the merge kernel may start taking SMs now
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kLmTmemCols) : "memory");
    }
}

// One CTA per (sequence, row): merges the row's per-tile statistics and stores the row statistics;
// the CTA that completes a sequence (arrival counter) runs the accept / first-rejection scan
// (Algorithm 6, for-loop).
template <bool GREEDY>
__global__ void __launch_bounds__(kThreads) lmhead_finalize_kernel(const VerifyParams p, const float2* lm_partial,
                                                                   const int NT) {
    __shared__ float2 s_w[kWarps];
    pdl_enter();
    const int b = blockIdx.x / p.R, lr = blockIdx.x - b * p.R;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = clamp_gamma(p.gamma[b], p.Gmax);
    const int rows_b = GREEDY ? g + 1 : 2 * g + 1;
    if (lr >= rows_b) return;
    const int r = row_slot(lr, g, p.Gmax);
    const float2* pp = lm_partial + ((size_t)b * p.R + r) * NT;
    float2 wr;
    if (GREEDY) {
        ArgMax a{-INFINITY, INT_MAX};
        for (int q = tid; q < NT; q += kThreads) {
            const float2 v = __ldcg(pp + q);
            a = better(a, ArgMax{v.x, __float_as_int(v.y)});
        }
        a = warp_best(a);
        wr = make_float2(a.m, __int_as_float(a.idx));
    } else {
        Online o{-INFINITY, 0.f};
        for (int q = tid; q < NT; q += kThreads) {
            const float2 v = __ldcg(pp + q);
            o.merge(v.x, v.y, p.c);
        }
        wr = warp_merge(o, p.c);
    }
    if (lane == 0) s_w[warp] = wr;
    __syncthreads();
    if (warp != 0) return;
    float2 st;
    if (GREEDY) {
        ArgMax a{-INFINITY, INT_MAX};
        if (lane < kWarps) a = ArgMax{s_w[lane].x, __float_as_int(s_w[lane].y)};
        a = warp_best(a);
        if (a.idx == INT_MAX) a.idx = 0;                      // row of -inf / NaN only
        st = make_float2(a.m, __int_as_float(a.idx));
    } else {
        Online o{-INFINITY, 0.f};
        if (lane < kWarps) { o.m = s_w[lane].x; o.s = s_w[lane].y; }
        st = warp_merge(o, p.c);
    }
    unsigned old = 0;
    if (lane == 0) {
        p.row_stats[(size_t)b * p.R + r] = st;
        __threadfence();
        old = atomicAdd(p.ticket + b, 1u);
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old + 1u == (unsigned)rows_b) {
        __threadfence();
        const float2* rsb = p.row_stats + (size_t)b * p.R;
        accept_scan_warp<float, GREEDY>(p, b, [rsb](int rr) { return __ldcg(rsb + rr); });
        if (lane == 0) p.ticket[b] = 0u;                      // leave the counter clear for the next call
    }
}

// ---- host side ------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

// bf16 matrix [rows, cols] with cols contiguous; boxes of box_rows x 64 columns, 128-byte swizzle,
// elements outside the matrix read as zero.
static bool make_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 matrix [rows, cols] with cols contiguous, written in boxes of 32 x 32 with the 128-byte swizzle
static bool make_out_map(CUtensorMap* tm, void* base, uint64_t rows, uint64_t cols) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

constexpr int kLmBN = 256;
constexpr size_t lm_smem_bytes(int mh, int stages) {
    return (size_t)stages * (mh * kLmABytes + (kLmBN / 64) * kLmChunkBytes) + kLmOutBytes + 1024;
}

static size_t lm_partial_bytes(int B, int Gmax, int V) {
    return align_up(sizeof(float2) * (size_t)B * (2 * Gmax + 1) * 2 * div_up(V, kLmBN), 256);
}

static std::atomic<bool> g_lm_attr[4][64];

template <int MH, int STAGES, bool GREEDY>
static bs_status launch_lmhead(const CUtensorMap* tms, const LmParams& lp, const VerifyParams& vp,
                               const float2* partial, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    auto kern = lmhead_gemm_kernel<kLmBN, MH, STAGES, GREEDY>;
    constexpr size_t smem = lm_smem_bytes(MH, STAGES);
    const int variant = (MH - 1) * 2 + (GREEDY ? 1 : 0);
    if (!g_lm_attr[variant][dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return cuda_status(cudaGetLastError());
        g_lm_attr[variant][dev] = true;
    }
    const int tiles = lp.prod[0].MT * lp.NT + (lp.nprod > 1 ? lp.prod[1].MT * lp.NT : 0);
    int grid = sm_count();
    if (grid > tiles) grid = tiles;
    cudaError_t e = launch_pdl(kern, grid, kLmThreads, smem, st, tms[0], tms[1], tms[2], tms[3], tms[4], tms[5], lp);
    if (e != cudaSuccess) return cuda_status(e);
    return cuda_status(launch_pdl(lmhead_finalize_kernel<GREEDY>, vp.B * vp.R, kThreads, 0, st, vp, partial, 2 * lp.NT));
}

}  // namespace bs

using namespace bs;

extern "C" size_t bs_lmhead_workspace_bytes(int B, int Gmax, int V) {
    const size_t base = bs_workspace_bytes(B, Gmax, V);
    if (!base) return 0;
    return align_up(base, 256) + lm_partial_bytes(B, Gmax, V);
}

extern "C" bs_status bs_lmhead_verify(const void* H_t, const void* W_t, int d_t, const void* H_d, const void* W_d,
                                      int d_d, const int32_t* draft_tokens, const int32_t* gamma,
                                      const float* u_accept, float temperature, int B, int Gmax, int V,
                                      float* logits_t_out, float* logits_d_out, int32_t* accept_len, float* p_tok,
                                      float* q_tok, void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 1 || Gmax < 0 || V < 1 || d_t < 1) return BS_ERR_INVALID_ARG;
    if (B > BS_MAX_BATCH || Gmax > BS_MAX_GAMMA || V > BS_MAX_VOCAB) return BS_ERR_UNSUPPORTED;
    if (!(temperature >= 0.f) || !isfinite(temperature)) return BS_ERR_INVALID_ARG;
    const bool greedy = temperature == 0.f;
    const bool need_draft = !greedy && Gmax > 0;
    if (!H_t || !W_t || !gamma || !logits_t_out || !accept_len || !workspace) return BS_ERR_INVALID_ARG;
    if (Gmax > 0 && !draft_tokens) return BS_ERR_INVALID_ARG;
    if (need_draft && (!H_d || !W_d || d_d < 1 || !logits_d_out || !u_accept)) return BS_ERR_INVALID_ARG;
    // tensor maps need 16-byte aligned bases and row pitches; the epilogue stores 16 bytes at a time
    if ((V % 8) || (d_t % 8) || (need_draft && (d_d % 8))) return BS_ERR_UNSUPPORTED;
    uintptr_t al = reinterpret_cast<uintptr_t>(H_t) | reinterpret_cast<uintptr_t>(W_t) |
                   reinterpret_cast<uintptr_t>(logits_t_out);
    if (need_draft)
        al |= reinterpret_cast<uintptr_t>(H_d) | reinterpret_cast<uintptr_t>(W_d) | reinterpret_cast<uintptr_t>(logits_d_out);
    if (al & 15) return BS_ERR_INVALID_ARG;
    const Workspace w = workspace_layout(B, Gmax, V);
    const size_t part_off = align_up(w.total, 256);
    if (workspace_bytes < part_off + lm_partial_bytes(B, Gmax, V) || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return BS_ERR_WORKSPACE;

    char* ws = static_cast<char*>(workspace);
    float2* partial = reinterpret_cast<float2*>(ws + part_off);

    LmParams lp;
    lp.nprod = need_draft ? 2 : 1;
    lp.V = V; lp.NT = div_up(V, kLmBN); lp.R = w.R;
    lp.c = greedy ? 1.f : kLog2e / temperature;
    lp.partial = partial;
    lp.abort_flag = reinterpret_cast<int32_t*>(ws + w.off_abort);
    const int Mt = B * (Gmax + 1), Md = B * Gmax;
    const int mh = Mt > kLmBM ? 2 : 1;                 // 256-row tiles once there is more than one row tile
    lp.prod[0] = LmProduct{logits_t_out, Mt, div_up(d_t, kLmBK), div_up(Mt, kLmBM * mh), Gmax + 1, 0};
    lp.prod[1] = LmProduct{logits_d_out, need_draft ? Md : 0, need_draft ? div_up(d_d, kLmBK) : 0,
                           need_draft ? div_up(Md, kLmBM * mh) : 0, Gmax > 0 ? Gmax : 1, Gmax + 1};

    CUtensorMap tms[6];
    if (!make_map(&tms[0], H_t, (uint64_t)Mt, (uint64_t)d_t, kLmBM) || !make_map(&tms[1], W_t, (uint64_t)d_t, (uint64_t)V, kLmBK))
        return BS_ERR_CUDA;
    if (need_draft) {
        if (!make_map(&tms[2], H_d, (uint64_t)Md, (uint64_t)d_d, kLmBM) || !make_map(&tms[3], W_d, (uint64_t)d_d, (uint64_t)V, kLmBK))
            return BS_ERR_CUDA;
    } else {
        tms[2] = tms[0];
        tms[3] = tms[1];
    }
    if (!make_out_map(&tms[4], logits_t_out, (uint64_t)Mt, (uint64_t)V)) return BS_ERR_CUDA;
    if (need_draft) {
        if (!make_out_map(&tms[5], logits_d_out, (uint64_t)Md, (uint64_t)V)) return BS_ERR_CUDA;
    } else {
        tms[5] = tms[4];
    }

    VerifyParams vp;
    vp.target = logits_t_out; vp.draft = logits_d_out; vp.tokens = draft_tokens; vp.gamma = gamma;
    vp.u_accept = u_accept; vp.accept_len = accept_len; vp.p_tok = p_tok; vp.q_tok = q_tok;
    vp.ticket = reinterpret_cast<uint32_t*>(ws + w.off_ticket_verify);
    vp.ticket_row = reinterpret_cast<uint32_t*>(ws + w.off_ticket_row);
    vp.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    vp.abort_flag = lp.abort_flag;
    vp.row_stats = reinterpret_cast<float2*>(ws + w.off_row_stats);
    vp.partial = reinterpret_cast<float2*>(ws + w.off_partial);
    vp.B = B; vp.Gmax = Gmax; vp.V = V; vp.R = w.R; vp.S = w.S;
    vp.seg = seg_elems(BS_F32); vp.nseg = div_up(V, vp.seg);
    vp.c = lp.c;
    vp.mode = kModeVerify; vp.position = 0; vp.draft_ready = vp.ticket_row; vp.draft_out = nullptr;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mh == 1)
        return greedy ? launch_lmhead<1, 4, true>(tms, lp, vp, partial, st)
                      : launch_lmhead<1, 4, false>(tms, lp, vp, partial, st);
    return greedy ? launch_lmhead<2, 3, true>(tms, lp, vp, partial, st) : launch_lmhead<2, 3, false>(tms, lp, vp, partial, st);
}
