// Arm selection and statistics update for B independent bandits, on the device so that a
// decoding round never returns to the host: UCBSpec (Algorithm 4 / Algorithm 8 of the paper)
// and EXP3Spec (Algorithm 5 / Algorithm 9), plus UCBSpec on a real-valued reward (Section 6.2:
// the throughput of the round).  The history H_t is kept as its sufficient statistics.  All index arithmetic is fp64 with explicit (non-fused) multiplies and adds.
//
// State blob (device memory owned by the caller):
//   [0, 256)  Header
//   A  [B, K] 8-byte: UCBSpec n_i (int64)         | EXP3Spec S_i = sum of loss estimates (fp64)
//   Bm [B, K] 8-byte: UCBSpec sum of rewards (int64) | EXP3Spec pulls per arm (int64, a statistic only)
//             real-reward UCBSpec: A = n_i (int64), Bm = sum of rewards (fp64)
//   t  [B] int64  completed rounds
//   ps [B] fp64   EXP3Spec: probability of the arm chosen by the pending select
#include "bs_common.cuh"

namespace bs {

struct BanditHeader {
    int alg, B, K, L;
    double delta;
    int arm_gamma[BS_MAX_ARMS];
    double width;        // real-reward UCBSpec: rewards live in [0, width]
};
static_assert(sizeof(BanditHeader) <= 256, "header must fit its slot");

struct BanditState {
    BanditHeader* hdr;
    long long* A_i;      // aliases A_d
    double* A_d;
    long long* Bm;
    double* Bm_d;        // aliases Bm
    long long* t;
    double* ps;
};

__host__ __device__ inline size_t bandit_bytes(int B, int K) {
    return 256 + align_up(sizeof(double) * (size_t)B * K, 256) * 2 + align_up(sizeof(double) * (size_t)B, 256) * 2;
}

__host__ __device__ inline BanditState bandit_view(void* state, int B, int K) {
    char* s = static_cast<char*>(state);
    BanditState v;
    v.hdr = reinterpret_cast<BanditHeader*>(s);
    size_t o = 256;
    v.A_i = reinterpret_cast<long long*>(s + o);
    v.A_d = reinterpret_cast<double*>(s + o);
    o += align_up(sizeof(double) * (size_t)B * K, 256);
    v.Bm = reinterpret_cast<long long*>(s + o);
    v.Bm_d = reinterpret_cast<double*>(s + o);
    o += align_up(sizeof(double) * (size_t)B * K, 256);
    v.t = reinterpret_cast<long long*>(s + o);
    o += align_up(sizeof(double) * (size_t)B, 256);
    v.ps = reinterpret_cast<double*>(s + o);
    return v;
}

// cr_{i,t} = (L/2) sqrt( (1+n)/n^2 * (1 + 2 ln( K t^2 sqrt(1+n) / delta )) )
// `half_width`: L/2 for the accepted length, W/2 for a reward in [0, W]
__device__ inline double confidence_radius(double half_width, int K, long long t, long long n, double delta) {
    const double n1 = __dadd_rn(1.0, (double)n);
    const double arg = __ddiv_rn(__dmul_rn((double)(K * t * t), sqrt(n1)), delta);
    const double inner = __dadd_rn(1.0, __dmul_rn(2.0, log(arg)));
    const double frac = __ddiv_rn(n1, (double)(n * n));
    return __dmul_rn(half_width, sqrt(__dmul_rn(frac, inner)));
}

// The select step for sequence b by one warp, lane i = arm i.
__device__ __forceinline__ void bandit_select_warp(const BanditState& s, int alg, int b, int K, const float* u_arm,
                                                   const uint8_t* active, int32_t* arm_out, int32_t* gamma_out,
                                                   double* index_out) {
    const int lane = threadIdx.x & 31;
    if (active && !active[b]) {
        if (lane == 0) { arm_out[b] = -1; gamma_out[b] = 0; }
        if (index_out && lane < K) index_out[(size_t)b * K + lane] = nan("");
        return;
    }
    const int L = s.hdr->L;
    const long long t = s.t[b];
    int arm;
    double shown = nan("");
    if (alg == BS_UCB || alg == BS_UCB_REWARD) {
        if (t < K) {
            arm = (int)t;                                   // rounds 1..K: arms 1..K in order
        } else {
            double idx = -INFINITY;
            if (lane < K) {
                const long long n = s.A_i[(size_t)b * K + lane];
                const double sum = alg == BS_UCB ? (double)s.Bm[(size_t)b * K + lane] : s.Bm_d[(size_t)b * K + lane];
                const double half = alg == BS_UCB ? __ddiv_rn((double)L, 2.0) : __ddiv_rn(s.hdr->width, 2.0);
                idx = n > 0 ? __dadd_rn(__ddiv_rn(sum, (double)n), confidence_radius(half, K, t, n, s.hdr->delta))
                            : INFINITY;
                shown = idx;
            }
            int best = lane;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double oi = __shfl_xor_sync(0xffffffffu, idx, o);
                const int ob = __shfl_xor_sync(0xffffffffu, best, o);
                if (oi > idx || (oi == idx && ob < best)) { idx = oi; best = ob; }   // ties: lowest arm
            }
            arm = best;
        }
    } else {
        // p_i proportional to exp(-eta_t * S_i), eta_t = sqrt(ln K / (t K)), t = this round's index
        const double eta = sqrt(__ddiv_rn(log((double)K), (double)((t + 1) * K)));
        const double Si = lane < K ? s.A_d[(size_t)b * K + lane] : INFINITY;
        double mn = Si;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        const double w = lane < K ? exp(__dmul_rn(-eta, __dadd_rn(Si, -mn))) : 0.0;
        double tot = 0.0;
        for (int i = 0; i < K; ++i) tot = __dadd_rn(tot, __shfl_sync(0xffffffffu, w, i));   // arm order
        const double pi = __ddiv_rn(w, tot);
        shown = pi;
        const double u = (double)u_arm[b];
        double c = 0.0, psel = 0.0;
        arm = -1;
        for (int i = 0; i < K; ++i) {
            const double p = __shfl_sync(0xffffffffu, pi, i);
            c = __dadd_rn(c, p);
            if (arm < 0 && (c > u || i == K - 1)) { arm = i; psel = p; }
        }
        if (lane == 0) s.ps[b] = psel;
    }
    if (lane == 0) {
        arm_out[b] = arm;
        gamma_out[b] = s.hdr->arm_gamma[arm];
    }
    if (index_out && lane < K) index_out[(size_t)b * K + lane] = shown;
}

// One warp per sequence.
__global__ void __launch_bounds__(128) bandit_select_kernel(void* state, int alg, int B, int K,
                                                           const float* u_arm, const uint8_t* active,
                                                           int32_t* arm_out, int32_t* gamma_out, double* index_out) {
    pdl_enter();
    const int b = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (b >= B) return;
    bandit_select_warp(bandit_view(state, B, K), alg, b, K, u_arm, active, arm_out, gamma_out, index_out);
}

// The history step for sequence b by one thread: accepted length y (UCBSpec, EXP3Spec) or real reward r.
__device__ __forceinline__ void bandit_update_one(const BanditState& s, int alg, int b, int K, const int32_t* arm,
                                                  const int32_t* reward_y, const double* reward_r,
                                                  const uint8_t* active) {
    if (active && !active[b]) return;
    const int a = arm[b];
    if (a < 0 || a >= K) return;
    if (alg == BS_UCB_REWARD) {
        double r = reward_r[b];
        r = isnan(r) ? 0.0 : fmin(fmax(r, 0.0), s.hdr->width);
        s.A_i[(size_t)b * K + a] += 1;
        s.Bm_d[(size_t)b * K + a] = __dadd_rn(s.Bm_d[(size_t)b * K + a], r);
    } else {
        const int L = s.hdr->L;
        const int y = max(1, min(reward_y[b], L + 1));      // accepted length, bonus included
        if (alg == BS_UCB) {
            s.A_i[(size_t)b * K + a] += 1;
            s.Bm[(size_t)b * K + a] += y;
        } else {
            // loss estimate (L + 1 - y) / (L p_{t, I_t}); the other arms' estimates are zero
            const double z = __ddiv_rn((double)(L + 1 - y), __dmul_rn((double)L, s.ps[b]));
            s.A_d[(size_t)b * K + a] = __dadd_rn(s.A_d[(size_t)b * K + a], z);
            s.Bm[(size_t)b * K + a] += 1;
        }
    }
    s.t[b] += 1;
}

__global__ void bandit_update_kernel(void* state, int alg, int B, int K, const int32_t* arm,
                                     const int32_t* reward_y, const double* reward_r, const uint8_t* active) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    bandit_update_one(bandit_view(state, B, K), alg, b, K, arm, reward_y, reward_r, active);
}

// History step of this round and select step of the next in one launch: one warp per sequence, lane 0
// records the outcome, then the warp chooses the next arm from the updated statistics.
__global__ void __launch_bounds__(128) bandit_step_kernel(void* state, int alg, int B, int K, const int32_t* reward_y,
                                                         const double* reward_r, const float* u_arm_next,
                                                         const uint8_t* active, int32_t* arm, int32_t* gamma,
                                                         double* index_out) {
    pdl_enter();
    const int b = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (b >= B) return;
    const BanditState s = bandit_view(state, B, K);
    if ((threadIdx.x & 31) == 0) bandit_update_one(s, alg, b, K, arm, reward_y, reward_r, active);
    __syncwarp();                                             // the lanes read what lane 0 wrote
    bandit_select_warp(s, alg, b, K, u_arm_next, active, arm, gamma, index_out);
}

// Tokens per second of the round: per sequence, or the batch total for every active sequence.
// One CTA; the total is an integer sum, so its order does not matter.
__global__ void __launch_bounds__(1024) throughput_reward_kernel(const int32_t* out_len, const uint8_t* active, int B,
                                                                 double seconds, int whole_batch, double* reward) {
    __shared__ unsigned long long s_total;
    pdl_enter();
    if (threadIdx.x == 0) s_total = 0ull;
    __syncthreads();
    if (whole_batch) {
        unsigned long long mine = 0ull;
        for (int b = threadIdx.x; b < B; b += blockDim.x)
            if (!active || active[b]) mine += (unsigned long long)max(out_len[b], 0);
        if (mine) atomicAdd(&s_total, mine);
        __syncthreads();
    }
    const double shared_r = __ddiv_rn((double)s_total, seconds);
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        double r = 0.0;
        if (!active || active[b]) r = whole_batch ? shared_r : __ddiv_rn((double)max(out_len[b], 0), seconds);
        reward[b] = r;
    }
}

}  // namespace bs

using namespace bs;

static bool bandit_args_ok(const void* state, size_t state_bytes, int alg, int B, int K) {
    return state && (alg == BS_UCB || alg == BS_EXP3 || alg == BS_UCB_REWARD) && B >= 1 && B <= BS_MAX_BATCH && K >= 1 && K <= BS_MAX_ARMS &&
           state_bytes >= bandit_bytes(B, K) && (reinterpret_cast<uintptr_t>(state) & 255) == 0;
}

extern "C" size_t bs_bandit_state_bytes(bs_alg alg, int B, int K) {
    if ((alg != BS_UCB && alg != BS_EXP3 && alg != BS_UCB_REWARD) || B < 1 || B > BS_MAX_BATCH || K < 1 || K > BS_MAX_ARMS) return 0;
    return bandit_bytes(B, K);
}

static bs_status bandit_init(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                             const int32_t* arm_gamma_host, double delta, double width, void* stream);

extern "C" bs_status bs_bandit_init_reward(void* state, size_t state_bytes, int B, int K,
                                           const int32_t* arm_gamma_host, double delta, double reward_width,
                                           void* stream) {
    if (!(reward_width > 0.0) || isinf(reward_width)) return BS_ERR_INVALID_ARG;
    return bandit_init(state, state_bytes, BS_UCB_REWARD, B, K, arm_gamma_host, delta, reward_width, stream);
}

extern "C" bs_status bs_bandit_init(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                                    const int32_t* arm_gamma_host, double delta, void* stream) {
    if (alg == BS_UCB_REWARD) return BS_ERR_INVALID_ARG;    // needs the reward range: bs_bandit_init_reward
    return bandit_init(state, state_bytes, alg, B, K, arm_gamma_host, delta, 0.0, stream);
}

static bs_status bandit_init(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                             const int32_t* arm_gamma_host, double delta, double width, void* stream) {
    if (!bandit_args_ok(state, state_bytes, alg, B, K) || !arm_gamma_host) return BS_ERR_INVALID_ARG;
    if (alg != BS_EXP3 && !(delta > 0.0)) return BS_ERR_INVALID_ARG;
    BanditHeader h;
    h.alg = alg; h.B = B; h.K = K; h.L = 0; h.delta = delta; h.width = width;
    for (int i = 0; i < BS_MAX_ARMS; ++i) h.arm_gamma[i] = 0;
    for (int i = 0; i < K; ++i) {
        if (arm_gamma_host[i] < 0 || arm_gamma_host[i] > BS_MAX_GAMMA) return BS_ERR_INVALID_ARG;
        h.arm_gamma[i] = arm_gamma_host[i];
        if (arm_gamma_host[i] > h.L) h.L = arm_gamma_host[i];
    }
    if (h.L < 1 && alg != BS_UCB_REWARD) return BS_ERR_INVALID_ARG;   // the radius and the loss estimate divide by L
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(state, 0, bandit_bytes(B, K), st);
    // pageable host source: the copy is staged before the call returns, so `h` may go out of scope
    if (e == cudaSuccess) e = cudaMemcpyAsync(state, &h, sizeof(h), cudaMemcpyHostToDevice, st);
    return cuda_status(e);
}

extern "C" bs_status bs_bandit_select(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                                      const float* u_arm, const uint8_t* active,
                                      int32_t* arm, int32_t* gamma, double* index_out, void* stream) {
    if (!bandit_args_ok(state, state_bytes, alg, B, K) || !arm || !gamma) return BS_ERR_INVALID_ARG;
    if (alg == BS_EXP3 && !u_arm) return BS_ERR_INVALID_ARG;
    const int warps_per_cta = 4;
    return cuda_status(launch_pdl(bandit_select_kernel, div_up(B, warps_per_cta), warps_per_cta * 32, 0,
                                  static_cast<cudaStream_t>(stream), state, (int)alg, B, K, u_arm, active, arm, gamma,
                                  index_out));
}

extern "C" bs_status bs_bandit_update(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                                      const int32_t* arm, const int32_t* reward_y, const uint8_t* active,
                                      void* stream) {
    if (!bandit_args_ok(state, state_bytes, alg, B, K) || !arm || !reward_y) return BS_ERR_INVALID_ARG;
    if (alg == BS_UCB_REWARD) return BS_ERR_INVALID_ARG;    // real rewards: bs_bandit_update_reward
    return cuda_status(launch_pdl(bandit_update_kernel, div_up(B, 128), 128, 0, static_cast<cudaStream_t>(stream),
                                  state, (int)alg, B, K, arm, reward_y, static_cast<const double*>(nullptr), active));
}

extern "C" bs_status bs_bandit_update_reward(void* state, size_t state_bytes, int B, int K,
                                             const int32_t* arm, const double* reward, const uint8_t* active,
                                             void* stream) {
    if (!bandit_args_ok(state, state_bytes, BS_UCB_REWARD, B, K) || !arm || !reward) return BS_ERR_INVALID_ARG;
    return cuda_status(launch_pdl(bandit_update_kernel, div_up(B, 128), 128, 0, static_cast<cudaStream_t>(stream),
                                  state, (int)BS_UCB_REWARD, B, K, arm, static_cast<const int32_t*>(nullptr), reward,
                                  active));
}

extern "C" bs_status bs_bandit_step(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                                    const int32_t* reward_y, const double* reward_r, const float* u_arm_next,
                                    const uint8_t* active, int32_t* arm, int32_t* gamma, double* index_out,
                                    void* stream) {
    if (!bandit_args_ok(state, state_bytes, alg, B, K) || !arm || !gamma) return BS_ERR_INVALID_ARG;
    if (alg == BS_UCB_REWARD ? !reward_r : !reward_y) return BS_ERR_INVALID_ARG;
    if (alg == BS_EXP3 && !u_arm_next) return BS_ERR_INVALID_ARG;
    const int warps_per_cta = 4;
    return cuda_status(launch_pdl(bandit_step_kernel, div_up(B, warps_per_cta), warps_per_cta * 32, 0,
                                  static_cast<cudaStream_t>(stream), state, (int)alg, B, K, reward_y, reward_r, u_arm_next,
                                  active, arm, gamma, index_out));
}

extern "C" bs_status bs_throughput_reward(const int32_t* out_len, const uint8_t* active, int B, double seconds,
                                          int whole_batch, double* reward, void* stream) {
    if (!out_len || !reward || B < 1 || B > BS_MAX_BATCH) return BS_ERR_INVALID_ARG;
    if (!(seconds > 0.0) || isinf(seconds)) return BS_ERR_INVALID_ARG;
    return cuda_status(launch_pdl(throughput_reward_kernel, 1, 1024, 0, static_cast<cudaStream_t>(stream), out_len,
                                  active, B, seconds, whole_batch ? 1 : 0, reward));
}

extern "C" bs_status bs_bandit_read(const void* state, size_t state_bytes, bs_alg alg, int B, int K,
                                    int64_t* n_host, int64_t* sumY_host, double* S_host, int64_t* t_host,
                                    void* stream) {
    if (!bandit_args_ok(state, state_bytes, alg, B, K)) return BS_ERR_INVALID_ARG;
    const BanditState s = bandit_view(const_cast<void*>(state), B, K);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    const size_t bk = sizeof(double) * (size_t)B * K;
    if (alg == BS_UCB) {
        if (n_host && e == cudaSuccess) e = cudaMemcpyAsync(n_host, s.A_i, bk, cudaMemcpyDeviceToHost, st);
        if (sumY_host && e == cudaSuccess) e = cudaMemcpyAsync(sumY_host, s.Bm, bk, cudaMemcpyDeviceToHost, st);
    } else if (alg == BS_UCB_REWARD) {
        if (n_host && e == cudaSuccess) e = cudaMemcpyAsync(n_host, s.A_i, bk, cudaMemcpyDeviceToHost, st);
        if (S_host && e == cudaSuccess) e = cudaMemcpyAsync(S_host, s.Bm_d, bk, cudaMemcpyDeviceToHost, st);
    } else {
        if (S_host && e == cudaSuccess) e = cudaMemcpyAsync(S_host, s.A_d, bk, cudaMemcpyDeviceToHost, st);
        if (n_host && e == cudaSuccess) e = cudaMemcpyAsync(n_host, s.Bm, bk, cudaMemcpyDeviceToHost, st);
    }
    if (t_host && e == cudaSuccess) e = cudaMemcpyAsync(t_host, s.t, sizeof(int64_t) * B, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return cuda_status(e);
}
