/*
 * banditspec.h -- C ABI of the B200 (sm_100a) library for one batched round of
 * speculative decoding with a bandit-chosen speculation length.
 *
 * One round, per sequence b of a batch of B independent sequences:
 *
 *   bs_bandit_select    choose the arm (speculation length gamma_b) for this round
 *   bs_softmax_verify   softmax statistics of every target / draft row, accept test,
 *                       first-rejection scan  -> accept_len[b] = tau_b
 *   bs_residual_sample  resample one token from Norm([P - Q]_+) at the rejected position,
 *                       or the bonus token from P when all drafts passed -> out_tokens, out_len
 *   bs_bandit_update    feed the accepted length y_b = tau_b + 1 back to the arm statistics
 *
 * plus bs_lmhead_verify, which computes the logits themselves (bf16 hidden states times
 * the bf16 output embedding on the tensor cores) fused with the softmax statistics.
 *
 * Conventions that hold for every entry point
 *  - Every array pointer is a DEVICE pointer owned by the caller unless the comment says
 *    "host".  The library allocates no device memory.  Its only process-wide state is a set of
 *    per-device values looked up on first use and never changed afterwards (the opt-in shared
 *    memory limit, kernel attributes, resident-CTA counts, the device address of the built-in
 *    scratch array of bs_softmax_verify_noalloc) and that scratch array itself; the values are
 *    held in atomics and every thread that finds one missing looks up the same answer, so calls
 *    may come from several host threads.
 *  - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous on that stream,
 *    never synchronise, and may be captured in a CUDA graph.
 *  - The return value covers host-side argument checks and launch errors only.  Problems
 *    found in device DATA (token id outside [0,V), gamma outside [0,Gmax], non-finite
 *    normaliser) are recorded per sequence in the workspace and read back with
 *    bs_get_device_status; the kernels never trap.
 *  - Row-major layouts with the vocabulary contiguous.  Row j (0-based) of either model is
 *    the distribution of drafted token j+1, i.e. conditioned on the prompt and the first j
 *    drafted tokens; target row gamma_b is the bonus position.  Padded entries (j >= gamma_b
 *    for tokens / uniforms / draft rows, j > gamma_b for target rows) are never read.
 *  - temperature > 0: sampling mode, probabilities are softmax(logits / temperature).
 *    temperature == 0: greedy mode (the limit of Section 2): a drafted token passes iff it
 *    equals the arg-max of its target row (lowest index among equal maxima); draft logits
 *    are not read and may be NULL.
 */
#ifndef BANDITSPEC_H_
#define BANDITSPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BS_OK = 0,
    BS_ERR_INVALID_ARG = 1,   /* NULL pointer, negative or unsupported size, bad enum */
    BS_ERR_CUDA = 2,          /* a CUDA runtime call or launch failed */
    BS_ERR_UNSUPPORTED = 3,   /* valid request outside the implemented limits */
    BS_ERR_WORKSPACE = 4,     /* workspace too small or misaligned */
    BS_ERR_TIMEOUT = 5,       /* bs_get_device_status: a bounded wait inside a kernel gave up */
    BS_ERR_DEVICE_DATA = 6    /* bs_get_device_status: some sequence carries a data error */
} bs_status;

typedef enum { BS_F32 = 0, BS_BF16 = 1 } bs_dtype;
typedef enum { BS_UCB = 0, BS_EXP3 = 1, BS_UCB_REWARD = 2 } bs_alg;

/* Per-sequence device status bits (bs_get_device_status). */
#define BS_DEV_BAD_GAMMA   1   /* gamma[b] outside [0, Gmax]; the sequence was processed as gamma = 0 */
#define BS_DEV_BAD_TOKEN   2   /* a drafted token outside [0, V); that position counts as rejected */
#define BS_DEV_NONFINITE   4   /* a softmax normaliser or residual mass was NaN / Inf / 0 */
#define BS_DEV_RESIDUAL_FALLBACK 8 /* [P-Q]_+ had zero mass at the rejected position; sampled from P instead */
#define BS_DEV_DRAFT_MISSING 16    /* bs_softmax_verify_drafted: a draft row below gamma_b was not produced by
                                      bs_draft_sample on this workspace; every draft of the sequence was rejected */
#define BS_DEV_BAD_TREE      32    /* bs_tree_verify_greedy: a node's parent is not an earlier node; the node counts as
                                      hanging under the prompt and never passes */

/* Limits of this implementation. */
#define BS_MAX_GAMMA   31      /* Gmax <= 31 (one warp scans the accept flags) */
#define BS_MAX_ARMS    32      /* K <= 32 (one lane per arm) */
#define BS_MAX_BATCH   4096    /* B <= 4096 */
#define BS_MAX_VOCAB   (1 << 20) /* V <= 1048576 */

const char* bs_status_string(bs_status s);

/* Text of the last CUDA runtime error that made a call on this thread return BS_ERR_CUDA
 * (diagnostics only; "no error" if there was none). */
const char* bs_last_cuda_error(void);

/* ---- workspace ------------------------------------------------------------------ */

/* Bytes of device scratch bs_softmax_verify / bs_residual_sample / bs_lmhead_verify need for
 * a batch of B sequences, speculation lengths up to Gmax and vocabulary V (any dtype).
 * Returns 0 for arguments outside the limits. */
size_t bs_workspace_bytes(int B, int Gmax, int V);

/* Clears the workspace (arrival counters must start at zero; the kernels leave them at zero
 * again after every call).  Call once after allocating, 256-byte aligned. */
bs_status bs_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Copies the per-sequence status words of the LAST verify/residual call to host memory.
 * Synchronises the stream.  host_status: host array [B].  Returns BS_ERR_DEVICE_DATA if any
 * word is non-zero, BS_ERR_TIMEOUT if a bounded wait inside a kernel of that call gave up (its
 * outputs are then undefined and its arrival counters may be left non-zero: clear the workspace
 * with bs_workspace_init before using it again), BS_OK otherwise. */
bs_status bs_get_device_status(const void* workspace, size_t workspace_bytes, int B, int Gmax, int V,
                               int32_t* host_status, void* stream);

/* ---- verification (Algorithm 6 of the paper, from its second line on) ---------------- */

/* Softmax statistics (Section 2: softmax of logits / temperature), accept test
 * r <= min{1, P(x)/Q(x)} and first-rejection scan (Algorithm 6, for-loop).
 *
 *  target_logits  [B, Gmax+1, V]  dtype
 *  draft_logits   [B, Gmax,   V]  dtype; may be NULL iff temperature == 0
 *  draft_tokens   [B, Gmax] int32, the drafted tokens x~_1..x~_gamma
 *  gamma          [B] int32, speculation length of each sequence this round, 0 <= gamma <= Gmax
 *  u_accept       [B, Gmax] fp32 uniforms in (0,1); may be NULL iff temperature == 0
 *  accept_len     [B] int32 out: tau_b = number of leading accepted drafts
 *  p_tok, q_tok   [B, Gmax] fp32 out or NULL: P_j(x~_{j+1}), Q_j(x~_{j+1}) for j < gamma_b
 *                 (entries j >= gamma_b are set to 0; both zero-filled in greedy mode).
 *                 Arithmetic is fp32 with the rounding of (row maximum * log2(e) / temperature)
 *                 undone to first order: measured error of a probability below 3e-7 for
 *                 temperatures from 0.05 to 8 at logits of +-10
 *  workspace      from bs_workspace_bytes / bs_workspace_init; keeps the row statistics that
 *                 bs_residual_sample reads, so the two calls share it and run on one stream.
 * Reads every valid logit exactly once.  Two calls that share a workspace must not overlap. */
bs_status bs_softmax_verify(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                            const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                            float temperature, int B, int Gmax, int V,
                            int32_t* accept_len, float* p_tok, float* q_tok,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Resampling step (Algorithm 6, else-branch and the line after the loop): for each sequence,
 * with tau = accept_len[b]: if tau < gamma_b sample from Norm([P_tau - Q_tau]_+), otherwise
 * sample the bonus token from P_gamma.  One uniform per sequence, inverse CDF in vocabulary
 * order: the smallest v whose cumulative mass strictly exceeds u * total.  Greedy mode emits
 * the arg-max of target row tau.
 *
 *  same logits / dtype / tokens / gamma / temperature / sizes / workspace as the preceding
 *  bs_softmax_verify call on this stream (its row statistics are read from the workspace)
 *  accept_len   [B] int32 in
 *  u_resample   [B] fp32 uniforms in (0,1); may be NULL iff temperature == 0
 *  out_tokens   [B, Gmax+1] int32 out: the tau accepted drafts, then the sampled token, then -1
 *  out_len      [B] int32 out: y_b = tau_b + 1, the accepted length that is the bandit reward
 *               (Section 3: the bonus token counts, 1 <= y <= L+1) */
bs_status bs_residual_sample(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                             const int32_t* draft_tokens, const int32_t* gamma, const int32_t* accept_len,
                             const float* u_resample, float temperature, int B, int Gmax, int V,
                             int32_t* out_tokens, int32_t* out_len,
                             void* workspace, size_t workspace_bytes, void* stream);

/* bs_softmax_verify without a caller-supplied workspace.  (No counterpart in the paper: this
 * exists for integration, not for the method.)
 *
 * For callers that cannot allocate device memory where the call is made: a decoding loop that
 * runs out of a pool sized at start-up, a plugin that only ever receives its input and output
 * buffers, or a latency-critical path where cudaMalloc is off limits because it synchronises the
 * device.  The scratch is a fixed array of BS_NOALLOC_SCRATCH_BYTES built into the library; every
 * GPU that loads the library holds that much memory until the process exits.
 *
 *  - Same arguments, outputs and arithmetic as bs_softmax_verify, minus the workspace.  The
 *    call allocates and frees nothing.
 *  - Limit: bs_workspace_bytes(B, Gmax, V) must not exceed BS_NOALLOC_SCRATCH_BYTES, otherwise
 *    BS_ERR_WORKSPACE is returned and nothing is launched (e.g. B=64, Gmax=8, V=128256 needs
 *    about 0.3 MB; B=256, Gmax=8, V=152064 about 1.4 MB).
 *  - The first call on each device looks up the device address of the array (with that device
 *    current).  Make that first call outside any stream capture.
 *  - All calls on a GPU share the one array.  It keeps what the previous call left; the counters
 *    and status words the kernel reads before writing are cleared on the stream at the start of
 *    every call.  Calls that overlap on the same GPU (different streams, different threads) race
 *    on it and give wrong results: serialise them.
 *  - The row statistics stay inside the library, so bs_residual_sample cannot follow this call;
 *    it serves callers that need accept_len and the token probabilities only.
 *  - The per-sequence status words and the abort word live in the array too, and
 *    bs_get_device_status cannot be pointed at it: device-detected data problems are handled as
 *    in bs_softmax_verify (an out-of-range token counts as rejected, an out-of-range gamma as
 *    gamma = 0, nothing traps) but are not reported, and a pipeline wait that gave up leaves
 *    accept_len / p_tok / q_tok of the unfinished sequences unwritten without a way to learn of
 *    it.  Callers that need the report use bs_softmax_verify with a workspace. */
#define BS_NOALLOC_SCRATCH_BYTES (2 << 20)
bs_status bs_softmax_verify_noalloc(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                    const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                    float temperature, int B, int Gmax, int V,
                                    int32_t* accept_len, float* p_tok, float* q_tok, void* stream);

/* ---- verification and resampling in one launch, with early exit ------------------------------- */

/* Algorithm 6 from its second line on in the algorithm's own order: position after position,
 * stopping at the first rejection (its "break"), then the resampling step -- bs_softmax_verify
 * followed by bs_residual_sample, but rows behind the first rejected draft are not needed: a
 * sequence that stops at position tau costs 2 (tau + 1) rows (2 gamma + 1 when everything
 * passes) plus a second pass over the rows of the stop position, instead of 2 gamma + 1 + 2.
 * (The kernel may stream a sequence up to three positions ahead of its last decision, so a few
 * rows behind the stop can be read all the same; they change no result.)
 *
 *  arguments as bs_softmax_verify and bs_residual_sample (temperature 0 = greedy mode: target rows
 *  only, the emitted token is the arg-max of the stop row, draft logits and uniforms may be NULL)
 *  p_tok, q_tok  [B, Gmax] fp32 out or NULL: filled for the positions that were examined
 *                (j <= tau_b, j < gamma_b); the entries behind the stop are set to 0 (all of them
 *                in greedy mode)
 *  accept_len, out_tokens, out_len: as the two separate calls
 * The CTAs that share a sequence wait for one another: they form a thread-block cluster, or --
 * rows of a single 32 KB segment, very large batches -- the kernel is launched cooperatively, and
 * the call fails with BS_ERR_CUDA where that is not possible.  A wait that does not end
 * within about a second makes bs_get_device_status return BS_ERR_TIMEOUT.
 * Requirement: rows on 16-byte boundaries (V * element size a multiple of 16, base pointers
 * 16-byte aligned), else BS_ERR_UNSUPPORTED. */
bs_status bs_verify_walk(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                         const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                         const float* u_resample, float temperature, int B, int Gmax, int V,
                         int32_t* accept_len, float* p_tok, float* q_tok, int32_t* out_tokens, int32_t* out_len,
                         void* workspace, size_t workspace_bytes, void* stream);

/* ---- drafting on the device (Algorithm 6, first line: x~_{j+1} ~ Q(. | pt, x~_{1:j})) ------------ */

/* Draws the drafted token of ONE position for every sequence that drafts it (position < gamma_b):
 * a categorical sample from softmax(draft row `position` / temperature) by inverse CDF in
 * vocabulary order with the uniform u_draft[b, position] (the smallest v whose cumulative mass
 * strictly exceeds u * total); at temperature 0 the arg-max of the row (lowest index among
 * equal maxima).  A draft model produces its rows one position at a time, so this is called once
 * per position, after the row has been written.
 *
 *  draft_logits [B, Gmax, V] dtype: only row `position` of each drafting sequence is read
 *  position     0 <= position < Gmax
 *  gamma        [B] int32: this round's speculation lengths
 *  u_draft      [B, Gmax] fp32 uniforms in (0,1); may be NULL iff temperature == 0
 *  draft_tokens [B, Gmax] int32: entry [b, position] is written for drafting sequences, others kept
 *  workspace    the round's verification workspace (bs_workspace_bytes / bs_workspace_init)
 * Besides the token, the call leaves the row's softmax statistics in the workspace and marks the
 * position as drafted, which is what bs_softmax_verify_drafted relies on.
 * Requirement: rows on 16-byte boundaries (V * element size a multiple of 16, base pointer
 * 16-byte aligned), else BS_ERR_UNSUPPORTED. */
bs_status bs_draft_sample(const void* draft_logits, bs_dtype dtype, int position, const int32_t* gamma,
                          const float* u_draft, float temperature, int B, int Gmax, int V,
                          int32_t* draft_tokens, void* workspace, size_t workspace_bytes, void* stream);

/* bs_softmax_verify for a round whose draft rows 0..gamma_b-1 all went through bs_draft_sample on
 * the same workspace: same arguments, outputs and arithmetic, but the draft rows are not streamed
 * again -- their statistics are taken from the workspace and only the logit of each drafted token
 * is read, so the call reads gamma_b + 1 rows per sequence instead of 2 gamma_b + 1.  A sequence
 * with an undrafted position below gamma_b gets accept_len = 0 and the status bit
 * BS_DEV_DRAFT_MISSING.  The drafted marks are consumed: the next round drafts again.
 * bs_residual_sample follows as after bs_softmax_verify.  Same alignment requirement as
 * bs_draft_sample. */
bs_status bs_softmax_verify_drafted(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                    const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                    float temperature, int B, int Gmax, int V,
                                    int32_t* accept_len, float* p_tok, float* q_tok,
                                    void* workspace, size_t workspace_bytes, void* stream);

/* bs_verify_walk for a round whose draft rows went through bs_draft_sample on the same workspace
 * (see bs_softmax_verify_drafted): only target rows are walked, position after position; of each
 * draft row the statistics left by drafting and the logit of the drafted token are used, and the
 * draft row of the stop position is read once for the residual.  Same arguments, outputs and
 * requirements as bs_verify_walk; an undrafted position stops the sequence there with
 * BS_DEV_DRAFT_MISSING; the drafted marks are consumed. */
bs_status bs_verify_walk_drafted(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                 const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                                 const float* u_resample, float temperature, int B, int Gmax, int V,
                                 int32_t* accept_len, float* p_tok, float* q_tok, int32_t* out_tokens,
                                 int32_t* out_len, void* workspace, size_t workspace_bytes, void* stream);

/* ---- greedy verification of a tree of drafted tokens (Section 3, example (2): the tree structure of
 *      the draft is the hyperparameter an arm stands for; Section 2: greedy decoding) -------------- */

/* The paper prints no verification rule for trees; at temperature -> 0 it is determined by Section 2
 * alone.  The target is a point mass on its arg-max, so the accept rule of Algorithm 6 accepts a drafted
 * token iff it IS the target's arg-max at its parent.  Node 0 is the prompt; node n = 1..n_b carries the
 * drafted token node_tokens[b, n-1] and hangs under node_parent[b, n-1], an earlier node (0..n-1).
 * Row n of target_logits[b] is the target's next-token distribution after the path to node n (what
 * a forward pass with tree attention returns), row 0 the one after the prompt.  A node passes iff its
 * parent passes (the prompt does) and its token is the arg-max of its parent's row (lowest index
 * among equal maxima).  The accepted path ends at the deepest passing node (the lowest-numbered one
 * among equally deep ones, which only matters if the draft repeated a token among siblings); the
 * arg-max of that node's own row is emitted after it.  Sampling mode is not offered for trees.
 *
 *  target_logits [B, Nmax+1, V] dtype; rows above n_b are never read
 *  node_parent   [B, Nmax] int32; node_tokens [B, Nmax] int32; n_nodes [B] int32, 0 <= n_b <= Nmax
 *  accept_len    [B] out: tau_b = depth of the node the accepted path ends at
 *  out_nodes     [B, Nmax] out or NULL: the nodes of the accepted path in order (the caller keeps
 *                their key/value entries), -1 behind it
 *  out_tokens    [B, Nmax+1] out: the accepted tokens, then the emitted arg-max, -1 behind it
 *  out_len       [B] out: y_b = tau_b + 1, the reward of the arm (Section 3)
 *  workspace     bs_workspace_bytes(B, Nmax, V) bytes; Nmax <= BS_MAX_GAMMA
 * Device-detected problems: n_b outside [0, Nmax] (BS_DEV_BAD_GAMMA, processed as the empty tree), a
 * token outside [0, V) (BS_DEV_BAD_TOKEN, the node never passes), a parent that is not an earlier
 * node (BS_DEV_BAD_TREE).  Two launches: the row-statistics kernel of bs_softmax_verify in greedy
 * mode (one arg-max per row, every valid logit read once) and a walk over the nodes. */
bs_status bs_tree_verify_greedy(const void* target_logits, bs_dtype dtype, const int32_t* node_parent,
                                const int32_t* node_tokens, const int32_t* n_nodes, int B, int Nmax, int V,
                                int32_t* accept_len, int32_t* out_nodes, int32_t* out_tokens, int32_t* out_len,
                                void* workspace, size_t workspace_bytes, void* stream);

/* Per-sequence trees from a table of K tree shapes (the arms): sequence b gets the parents and the node
 * count of shape arm[b], as bs_bandit_select chose it (arm[b] < 0, an inactive sequence: the empty tree).
 *  shape_parent [K, Nmax] int32, shape_nodes [K] int32, arm [B] int32 (all device)
 *  node_parent  [B, Nmax] out, n_nodes [B] out */
bs_status bs_tree_expand_shapes(const int32_t* shape_parent, const int32_t* shape_nodes, const int32_t* arm, int K,
                                int B, int Nmax, int32_t* node_parent, int32_t* n_nodes, void* stream);

/* ---- fused LM head (Algorithm 6, second line: the models are evaluated on all drafted positions
 *      in parallel; the last step of that evaluation is logits = H W) -------------------------- */

/* Bytes of device scratch bs_lmhead_verify needs.  The first bs_workspace_bytes(B, Gmax, V) bytes
 * are an ordinary verification workspace (clear it with bs_workspace_init before the first call),
 * so the same pointer and size are then handed to bs_residual_sample and bs_get_device_status.
 * Returns 0 for arguments outside the limits. */
size_t bs_lmhead_workspace_bytes(int B, int Gmax, int V);

/* Computes the target and draft logits from the final hidden states on the tensor cores
 * (bf16 x bf16 products, fp32 accumulation), the softmax statistics of every row while the
 * logits are still on chip, and then the accept test and first-rejection scan of
 * bs_softmax_verify.  The fp32 logits are written out so that
 *   bs_residual_sample(logits_t_out, logits_d_out, BS_F32, ..., workspace, ...)
 * can follow on the same stream.
 *
 *  H_t  [B * (Gmax+1), d_t] bf16, d_t contiguous: row b * (Gmax+1) + j is the target model's final
 *       hidden state at drafted position j of sequence b (j = Gmax is the bonus position)
 *  W_t  [d_t, V] bf16, V contiguous: the target model's output embedding
 *  H_d  [B * Gmax, d_d] bf16, W_d [d_d, V] bf16: the same for the draft model; all four may be
 *       NULL (and d_d 0) iff temperature == 0 or Gmax == 0
 *  logits_t_out [B, Gmax+1, V] fp32 out;  logits_d_out [B, Gmax, V] fp32 out (NULL iff no draft product)
 *  draft_tokens, gamma, u_accept, temperature, accept_len, p_tok, q_tok: as bs_softmax_verify
 *  workspace    at least bs_lmhead_workspace_bytes(B, Gmax, V) bytes, 256-byte aligned
 * Every row of H is multiplied, padded positions (j > gamma_b) included: they must be readable
 * and their logits are written, but they take no part in the verification.
 * Requirements: V, d_t and d_d multiples of 8; all matrix pointers 16-byte aligned; otherwise
 * BS_ERR_UNSUPPORTED / BS_ERR_INVALID_ARG.  A pipeline wait inside the kernel that does not
 * complete within about a second makes bs_get_device_status return BS_ERR_TIMEOUT. */
bs_status bs_lmhead_verify(const void* H_t, const void* W_t, int d_t, const void* H_d, const void* W_d, int d_d,
                           const int32_t* draft_tokens, const int32_t* gamma, const float* u_accept,
                           float temperature, int B, int Gmax, int V,
                           float* logits_t_out, float* logits_d_out,
                           int32_t* accept_len, float* p_tok, float* q_tok,
                           void* workspace, size_t workspace_bytes, void* stream);

/* ---- arm selection (Algorithm 3, select and history lines) ---------------------------- */

/* Bytes of the opaque device state of B independent bandits with K arms. 0 if out of limits. */
size_t bs_bandit_state_bytes(bs_alg alg, int B, int K);

/* Resets the state: no pulls, no rounds.  arm_gamma: HOST array [K], speculation length of
 * each arm; L = max_i arm_gamma[i] is the maximum speculation length of the configuration.
 * delta: confidence parameter of UCBSpec (Algorithm 4 input; the regret proof uses 1/2);
 * ignored by EXP3Spec.  The state is plain device memory: copying its bytes checkpoints it. */
bs_status bs_bandit_init(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                         const int32_t* arm_gamma_host, double delta, void* stream);

/* Chooses this round's arm for every active sequence.
 *  UCBSpec (Algorithm 4 / Algorithm 8): arm t in the first K rounds (t = completed rounds),
 *    then argmax_i  sumY_i/n_i + (L/2) sqrt((1+n_i)/n_i^2 (1 + 2 ln(K t^2 sqrt(1+n_i)/delta))),
 *    lowest index on ties.  u_arm is not read and may be NULL.
 *  EXP3Spec (Algorithm 5 / Algorithm 9): p_i proportional to exp(-eta_t S_i),
 *    eta_t = sqrt(ln K / (t K)) with t = completed rounds + 1; the arm is the smallest i whose
 *    cumulative probability strictly exceeds u_arm[b]; p of the chosen arm is kept for the update.
 *  u_arm   [B] fp32 uniforms in (0,1) (EXP3Spec)
 *  active  [B] uint8 or NULL (= all active); inactive sequences get arm = -1, gamma = 0
 *  arm     [B] int32 out;  gamma [B] int32 out = arm_gamma[arm]
 *  index_out [B, K] fp64 out or NULL: the UCB index values / EXP3 probabilities used (NaN
 *            during UCBSpec's round-robin prefix) -- for tests and logging. */
bs_status bs_bandit_select(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                           const float* u_arm, const uint8_t* active,
                           int32_t* arm, int32_t* gamma, double* index_out, void* stream);

/* Records the outcome of the round for every active sequence.
 *  UCBSpec: n[arm] += 1, sumY[arm] += y, t += 1.
 *  EXP3Spec: S[arm] += (L + 1 - y) / (L * p_arm), t += 1  (loss estimate of Algorithm 9).
 *  arm [B] int32 in (as returned by select); reward_y [B] int32 in, 1 <= y <= L+1
 *  (out_len of bs_residual_sample); values outside that range are clamped. */
bs_status bs_bandit_update(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                           const int32_t* arm, const int32_t* reward_y, const uint8_t* active,
                           void* stream);

/* bs_bandit_update of this round and bs_bandit_select of the next in one launch (Algorithm 3: the
 * history line of round t, then the select line of round t + 1), with the same results as the
 * two calls.
 *  reward_y [B] int32 (UCBSpec, EXP3Spec) or reward_r [B] fp64 (BS_UCB_REWARD): the other may be NULL
 *  u_arm_next [B] fp32: the uniforms of the next round's draw (EXP3Spec; else may be NULL)
 *  active: one mask for both steps (NULL = all active)
 *  arm [B] int32 in/out: the arms played this round on entry, the next round's arms on return
 *  gamma [B] int32 out: the next round's speculation lengths.  It must not be the array a kernel
 *  still in flight on another stream reads; on one stream the call is ordered like any other.
 *  index_out as in bs_bandit_select. */
bs_status bs_bandit_step(void* state, size_t state_bytes, bs_alg alg, int B, int K,
                         const int32_t* reward_y, const double* reward_r, const float* u_arm_next,
                         const uint8_t* active, int32_t* arm, int32_t* gamma, double* index_out,
                         void* stream);

/* Reads the sufficient statistics back to host arrays (any may be NULL).  Synchronises.
 *  UCBSpec: n_host [B,K] int64, sumY_host [B,K] int64, t_host [B] int64; S_host unused.
 *  EXP3Spec: S_host [B,K] fp64, n_host [B,K] int64 (pulls per arm, not used by the algorithm),
 *            t_host [B] int64; sumY_host unused. */
bs_status bs_bandit_read(const void* state, size_t state_bytes, bs_alg alg, int B, int K,
                         int64_t* n_host, int64_t* sumY_host, double* S_host, int64_t* t_host,
                         void* stream);

/* ---- throughput as the reward (Section 6.2) -------------------------------------------
 * Section 6.2 runs UCBSpec over the speculation lengths {0, ..., 4} (0 = canonical decoding,
 * Algorithm 1) with "the current throughput", generated tokens per second, as the reward, and
 * prints no formula.  Reading: alg = BS_UCB_REWARD is Algorithm 8 with the history holding
 * real rewards r in [0, W] and the radius factor L/2 (half the width of [1, L+1], where the
 * accepted length lives) replaced by W/2.  bs_bandit_state_bytes, bs_bandit_select and
 * bs_bandit_read take BS_UCB_REWARD; bs_bandit_init and bs_bandit_update do not (they return
 * BS_ERR_INVALID_ARG): use the two calls below.  bs_bandit_read: n_host [B,K] int64 pulls,
 * S_host [B,K] fp64 reward sums, t_host [B] int64; sumY_host unused. */

/* bs_bandit_init for BS_UCB_REWARD.  reward_width = W > 0, finite.  arm_gamma may be all
 * zero (L is not used by this algorithm). */
bs_status bs_bandit_init_reward(void* state, size_t state_bytes, int B, int K,
                                const int32_t* arm_gamma_host, double delta, double reward_width,
                                void* stream);

/* n[arm] += 1, sumR[arm] += r, t += 1 for every active sequence.
 *  arm [B] int32 device, as returned by select;  reward [B] fp64 device: values outside
 *  [0, W] are clamped into it, NaN counts as 0. */
bs_status bs_bandit_update_reward(void* state, size_t state_bytes, int B, int K,
                                  const int32_t* arm, const double* reward, const uint8_t* active,
                                  void* stream);

/* The round's throughput as a reward, on the device (fp64).
 *  out_len [B] int32 device: tokens sequence b emitted in the round (bs_residual_sample)
 *  seconds: HOST scalar > 0, finite: what the caller measured for the round
 *  whole_batch = 0: reward[b] = out_len[b] / seconds
 *  whole_batch = 1: reward[b] = (sum of out_len over the active sequences) / seconds for every
 *                   active b -- bandits that start together then stay together, so the batch
 *                   shares one speculation length, as one serving step does
 *  reward [B] fp64 device out; inactive sequences get 0. */
bs_status bs_throughput_reward(const int32_t* out_len, const uint8_t* active, int B, double seconds,
                               int whole_batch, double* reward, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BANDITSPEC_H_ */
