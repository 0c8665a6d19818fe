// bs_tree_verify_greedy: greedy verification of a TREE of drafted tokens -- the paper's second
// family of arms (Section 3, example (2): the hyperparameter of the speculative-decoding subroutine
// is the tree structure), at temperature -> 0 (Section 2: the next token is the one with the highest
// logit).  For a degenerate target the accept rule of Algorithm 6 accepts a drafted token iff it is the
// target's arg-max at its parent, so: a node passes iff its parent passes and its token is the arg-max
// of its parent's row (lowest index among equal maxima); the deepest passing node (lowest-numbered
// among equally deep ones) ends the accepted path, and the arg-max of its own row is emitted after it.
//
// The heavy part -- the arg-max of every row of every tree -- is the greedy mode of the row-statistics
// kernels, unchanged: the tree's nodes take the place of the drafted positions (row n = node n, row 0 =
// the prompt).  What is added is one small kernel, a warp per sequence, that turns the arg-maxes and the
// parent array into the accepted path.
#include "bs_verify_common.cuh"

namespace bs {

struct TreeParams {
    const int32_t* node_parent;   // [B, Nmax] parent of node n = 1..n_b at [n - 1], in [0, n - 1]; 0 = the prompt
    const int32_t* node_tokens;   // [B, Nmax]
    const int32_t* n_nodes;       // [B]
    const float2* row_stats;      // [B, R]: (max, arg-max bits) of rows 0..n_b, left by the statistics kernel
    int32_t* status;              // [B]
    int32_t* accept_len;          // [B]
    int32_t* out_nodes;           // [B, Nmax] or NULL
    int32_t* out_tokens;          // [B, Nmax + 1]
    int32_t* out_len;             // [B]
    int B, Nmax, V, R;
};

constexpr int kTreeWarps = 4;

__global__ void __launch_bounds__(kTreeWarps * 32) tree_walk_kernel(const TreeParams p) {
    pdl_enter();                                              // the arg-maxes come from the kernel before this one
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kTreeWarps + (threadIdx.x >> 5);
    if (b >= p.B) return;
    const int nraw = p.n_nodes[b];
    const int n = clamp_gamma(nraw, p.Nmax);                  // an out-of-range count is processed as an empty tree
    const float2* rs = p.row_stats + (size_t)b * p.R;
    // lane l holds node l + 1
    int par = 0, tok = -1, bits = 0;
    bool match = false;
    if (lane < n) {
        par = p.node_parent[(size_t)b * p.Nmax + lane];
        tok = p.node_tokens[(size_t)b * p.Nmax + lane];
        if (par < 0 || par > lane) {                          // a parent must come before its child
            bits |= BS_DEV_BAD_TREE;
            par = 0;
        } else {
            match = tok == __float_as_int(rs[par].y) && tok >= 0 && tok < p.V;
        }
    }
    // nodes in index order: a node passes iff its parent does and its token is the parent row's arg-max
    unsigned passes = 1u;                                     // bit n: node n passes; bit 0 = the prompt
    int depth = 0;                                            // of this lane's node
    for (int k = 1; k <= n; ++k) {
        const int kp = __shfl_sync(0xffffffffu, par, k - 1);
        const bool km = __shfl_sync(0xffffffffu, (int)match, k - 1) != 0;
        const int dp = kp == 0 ? 0 : __shfl_sync(0xffffffffu, depth, (kp - 1) & 31);
        if (lane == k - 1) depth = dp + 1;
        if (km && ((passes >> kp) & 1u)) passes |= 1u << k;   // k <= 31
    }
    // the deepest passing node, the lowest-numbered among equally deep ones
    int key = (lane < n && ((passes >> (lane + 1)) & 1u)) ? depth * 64 + (63 - (lane + 1)) : -1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
    const int best = key < 0 ? 0 : 63 - (key & 63);
    const int tau = key < 0 ? 0 : key >> 6;
    // walk back from it: position j of the path (0-based) is the ancestor at depth j + 1
    int32_t* ot = p.out_tokens + (size_t)b * (p.Nmax + 1);
    int32_t* on = p.out_nodes ? p.out_nodes + (size_t)b * p.Nmax : nullptr;
    int c = best;
    for (int j = tau - 1; j >= 0; --j) {
        const int ctok = __shfl_sync(0xffffffffu, tok, (c - 1) & 31);
        const int cpar = __shfl_sync(0xffffffffu, par, (c - 1) & 31);
        if (lane == 0) {
            ot[j] = ctok;
            if (on) on[j] = c;
        }
        c = cpar;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
    for (int j = tau + 1 + lane; j <= p.Nmax; j += 32) ot[j] = -1;
    if (on)
        for (int j = tau + lane; j < p.Nmax; j += 32) on[j] = -1;
    if (lane == 0) {
        ot[tau] = __float_as_int(rs[best].y);                 // the arg-max after the accepted path
        p.accept_len[b] = tau;
        p.out_len[b] = tau + 1;
        // the statistics kernel tested the nodes as if they were a chain and may have flagged tokens outside
        // the vocabulary; what it wrote is kept, the tree's own findings are added
        if (bits) p.status[b] |= bits;
    }
}

// Per-sequence trees from a table of shapes: sequence b gets shape arm[b] (an arm < 0, a sequence that
// sits the round out, gets the empty tree).
__global__ void tree_expand_kernel(const int32_t* shape_parent, const int32_t* shape_nodes, const int32_t* arm, int K,
                                   int B, int Nmax, int32_t* node_parent, int32_t* n_nodes) {
    pdl_enter();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * Nmax) return;
    const int b = i / Nmax, k = i - b * Nmax;
    const int a = arm[b];
    const bool ok = a >= 0 && a < K;
    node_parent[i] = ok ? shape_parent[(size_t)a * Nmax + k] : 0;
    if (k == 0) n_nodes[b] = ok ? shape_nodes[a] : 0;
}

}  // namespace bs

using namespace bs;

extern "C" bs_status bs_tree_verify_greedy(const void* target_logits, bs_dtype dtype, const int32_t* node_parent,
                                           const int32_t* node_tokens, const int32_t* n_nodes, int B, int Nmax, int V,
                                           int32_t* accept_len, int32_t* out_nodes, int32_t* out_tokens,
                                           int32_t* out_len, void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 1 || Nmax < 0 || V < 1) return BS_ERR_INVALID_ARG;
    if (!target_logits || !n_nodes || !accept_len || !out_tokens || !out_len || !workspace) return BS_ERR_INVALID_ARG;
    if (Nmax > 0 && (!node_parent || !node_tokens)) return BS_ERR_INVALID_ARG;
    // the arg-max of rows 0..n_b of every sequence: the statistics kernels in greedy mode, with the nodes in
    // place of the drafted positions (their chain-shaped accept test writes accept_len; the walk below overwrites it)
    const bs_status s = run_verify(target_logits, nullptr, dtype, node_tokens, n_nodes, nullptr, 0.f, B, Nmax, V,
                                   accept_len, nullptr, nullptr, workspace, workspace_bytes, stream, kModeVerify, 0, nullptr);
    if (s != BS_OK) return s;
    const Workspace w = workspace_layout(B, Nmax, V);
    char* ws = static_cast<char*>(workspace);
    TreeParams p;
    p.node_parent = node_parent; p.node_tokens = node_tokens; p.n_nodes = n_nodes;
    p.row_stats = reinterpret_cast<const float2*>(ws + w.off_row_stats);
    p.status = reinterpret_cast<int32_t*>(ws + w.off_status);
    p.accept_len = accept_len; p.out_nodes = out_nodes; p.out_tokens = out_tokens; p.out_len = out_len;
    p.B = B; p.Nmax = Nmax; p.V = V; p.R = w.R;
    return cuda_status(launch_pdl(tree_walk_kernel, div_up(B, kTreeWarps), kTreeWarps * 32, 0,
                                  static_cast<cudaStream_t>(stream), p));
}

extern "C" bs_status bs_tree_expand_shapes(const int32_t* shape_parent, const int32_t* shape_nodes, const int32_t* arm,
                                           int K, int B, int Nmax, int32_t* node_parent, int32_t* n_nodes, void* stream) {
    if (K < 1 || B < 1 || Nmax < 1 || Nmax > BS_MAX_GAMMA || B > BS_MAX_BATCH) return BS_ERR_INVALID_ARG;
    if (!shape_parent || !shape_nodes || !arm || !node_parent || !n_nodes) return BS_ERR_INVALID_ARG;
    return cuda_status(launch_pdl(tree_expand_kernel, div_up(B * Nmax, 256), 256, 0, static_cast<cudaStream_t>(stream),
                                  shape_parent, shape_nodes, arm, K, B, Nmax, node_parent, n_nodes));
}
