/*
 * mtad.h - C ABI of the MTAD / MMTAD verification hot path (arxiv 2407.09722) for NVIDIA B200 (sm_100a).
 *
 * One iteration of the method (Algorithm 1; Sec. 3.3 for the multi-candidate form) is
 *     draft with the auxiliary model  ->  one target forward over all draft rows  ->  joint likelihood of
 *     every draft prefix  ->  threshold test  ->  longest accepted prefix + one extra token from the target.
 * This library runs everything from the target forward on (mtad_verify_chain / mtad_verify_tree), the KV-cache
 * roll-forward that the paper calls the rollback operation (kv_commit), and the beam-sampling draft
 * (mtad_draft).  Every step executes in CUDA kernels of this library; there is no CPU fallback.
 *
 * Conventions
 *   - Every function returns an int status: MTAD_OK (0) or a negative MTAD_E_* code.  Nothing throws, exits
 *     or aborts.  mtad_status_str() names a code.
 *   - "device" pointers are CUDA device memory owned by the caller for the whole lifetime of the context;
 *     "host" pointers are ordinary memory read during the call only.  The library allocates no device memory:
 *     all scratch lives in the workspace the caller hands to mtad_create.
 *   - All device work is enqueued on the stream passed in (a cudaStream_t cast to void*; NULL = the legacy
 *     default stream) and the call returns without synchronising, unless stated otherwise.
 *   - Rows.  A verify call runs R = 1 + N rows per sequence: row 0 is the *root*, the last emitted token whose
 *     K/V are not yet cached (position L, the committed length); row n+1 is draft node n at position
 *     L + depth(n).  Row r writes its K/V to cache slot L + r.  A row attends to positions [0, L) and to the
 *     rows of its ancestors and itself (tree attention, Sec. 3.3).
 *   - Matrices are bf16, row-major [out_features, in_features].  Accumulation, norms, softmax and the residual
 *     stream are fp32.  The KV cache stores bf16.
 *   - A context is not thread-safe; use one context per stream.
 */
#ifndef MTAD_H_
#define MTAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    MTAD_OK = 0,
    MTAD_E_INVALID = -1,       /* bad argument: null pointer, size out of range, tau outside [0,1), NaN */
    MTAD_E_CAPACITY = -2,      /* batch, node count, depth or KV capacity exceeded */
    MTAD_E_CUDA = -3,          /* a CUDA call failed; mtad_last_cuda_error() gives the code */
    MTAD_E_TIMEOUT = -4,       /* a bounded device-side wait gave up (reported through the status words) */
    MTAD_E_UNIMPLEMENTED = -5,
    MTAD_E_WORKSPACE = -6      /* workspace missing, misaligned or too small */
};

#define MTAD_MAX_BATCH 64        /* sequences per call */
#define MTAD_MAX_NODES 255       /* draft nodes per sequence per call */
#define MTAD_MAX_DEPTH 32        /* deepest draft node */
#define MTAD_LAYER_TENSORS 9     /* attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down */

/* Bits of the per-sequence device status word (mtad_result.status), written by the kernels.  A sequence with
 * a non-zero status produced no valid result and its cache is not touched by kv_commit. */
#define MTAD_ST_BAD_PARENT   1u  /* parent[n] >= n or < -1 */
#define MTAD_ST_BAD_TOKEN    2u  /* token id outside [0, vocab) */
#define MTAD_ST_KV_OVERFLOW  4u  /* L + rows > kv_capacity */
#define MTAD_ST_TOO_DEEP     8u  /* depth > max_depth passed to the call */
#define MTAD_ST_BAD_COUNT   16u  /* n_nodes[b] outside [0, max_nodes] */
#define MTAD_ST_TIMEOUT     32u  /* a bounded wait inside a kernel gave up */
#define MTAD_ST_AUX_PENDING 64u  /* more than MTAD_MAX_DEPTH + 1 tokens wait to be replayed by the auxiliary model */
#define MTAD_ST_NONFINITE  128u  /* a row of target logits was not finite (NaN or infinite weights, cache or input) */
#define MTAD_ST_RANGE     256u  /* an index derived from device-resident state (length, slot, node id, path) fell
                                    outside its array: the access was skipped (corrupted state or a library bug) */
#define MTAD_MAX_BEAM 8          /* beam width of mtad_draft */

/* A Llama-style decoder (pre-RMSNorm, rotary embedding with half-split pairing (i, i + head_dim/2), grouped-
 * query attention scaled by 1/sqrt(head_dim), SwiGLU FFN, no biases, untied LM head).  The paper names model
 * families only (Sec. 5); this is the decoder its Llama pairs use. */
typedef struct mtad_model_desc {
    int32_t layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_base, rms_eps;
    const void* embed;                 /* device bf16 [vocab, d_model] */
    const void* lm_head;               /* device bf16 [vocab, d_model] */
    const void* final_norm;            /* device bf16 [d_model] */
    const void* const* layer_weights;  /* HOST array of layers * MTAD_LAYER_TENSORS device bf16 pointers, in the
                                          order attn_norm[d], wq[Hq*hd, d], wk[Hkv*hd, d], wv[Hkv*hd, d],
                                          wo[d, Hq*hd], ffn_norm[d], w_gate[F, d], w_up[F, d], w_down[d, F] */
    void* kv_cache;                    /* device bf16 [layers][max_batch][2 (K,V)][n_kv_heads][kv_capacity][head_dim];
                                          K is stored after the rotary embedding */
    int64_t kv_capacity;               /* positions per sequence */
} mtad_model_desc;

/* Outputs of a verify call; device arrays owned by the caller.  B = sequences in the call, N = max_nodes of the
 * call, D = max_depth of the call (chain: N = D = gamma).  Optional members may be NULL. */
typedef struct mtad_result {
    int32_t* eta;          /* [B]   accepted draft tokens (length of the winning path) */
    int32_t* winner;       /* [B]   node index of the accepted candidate, -1 = none (only the root is kept) */
    int32_t* path;         /* [B,D] node ids root-to-winner, first eta entries valid */
    int32_t* n_out;        /* [B]   eta + 1 */
    int32_t* out_tok;      /* [B,D+1] accepted tokens followed by the extra token drawn from the target */
    float*   out_lp;       /* [B,D+1] their target log-probabilities (conditional, per token) */
    float*   node_lp;      /* [B,N] log p(tok[n] | path to n), optional */
    float*   node_LP;      /* [B,N] joint log-likelihood of the path ending at n, optional */
    float*   row_lse;      /* [B,N+1] log-sum-exp of each row's logits, optional */
    int32_t* row_cand;     /* [B,N+1] Gumbel-argmax token of each row, optional */
    float*   row_cand_lp;  /* [B,N+1] its log-probability, optional */
    float*   margin;       /* [B,2] smallest |log p - log q - log tau| over the tested nodes; LP gap between the
                                    winner and the best other passing node of its depth (+inf if none), optional */
    uint32_t* status;      /* [B]   MTAD_ST_* bits, 0 = fine */
} mtad_result;

typedef struct mtad_ctx mtad_ctx;

/* Bytes of device workspace a context for these models needs.  aux may be NULL (no draft model). */
int mtad_workspace_bytes(const mtad_model_desc* target, const mtad_model_desc* aux, int max_batch, int max_nodes,
                         size_t* out_bytes);

/* Create a context.  workspace: device memory, 256-byte aligned, at least mtad_workspace_bytes(); it is zeroed
 * and the call synchronises the device.  The descriptors (and the host pointer arrays in them) are copied; the
 * device memory they point to stays the caller's.  All sequences start empty (L = 0, root token 0). */
int mtad_create(const mtad_model_desc* target, const mtad_model_desc* aux, int max_batch, int max_nodes,
                void* workspace, size_t workspace_bytes, mtad_ctx** out);
int mtad_destroy(mtad_ctx* ctx);

/* Set sequence `seq` to committed length kv_len (positions [0, kv_len) of the target cache are taken as valid,
 * e.g. injected by the caller) with `root_token` as the last emitted token.  kv_len = 0 starts a fresh sequence;
 * a prompt is then pushed as draft chains with log_tau = -INFINITY (tau = 0 accepts every prefix) and kv_commit.
 * aux_len is the committed length of the auxiliary cache (<= kv_len); the kv_len - aux_len tokens in between
 * (at most MTAD_MAX_DEPTH) are given in pending_tok (host; may be NULL when aux_len == kv_len) and are replayed
 * by the next mtad_draft. */
int mtad_seq_set(mtad_ctx* ctx, int seq, int32_t kv_len, int32_t root_token, int32_t aux_len,
                 const int32_t* pending_tok, void* stream);

/* Read back the committed length and root token of a sequence.  Synchronises the stream. */
int mtad_seq_get(mtad_ctx* ctx, int seq, int32_t* kv_len, int32_t* root_token, void* stream);

/* The context keeps, on the host, an upper bound of every sequence's committed length (it sizes the attention
 * launch and the capacity checks of mtad_draft without reading device memory).  kv_commit can only add the largest
 * possible advance (max_depth + 1) to it, so over a long decode loop the bound drifts above the true length.  A
 * caller that reads eta back anyway hands the true length in here (host-side, no launch, no synchronisation);
 * mtad_seq_get also refreshes the bound.  Without either, mtad_draft may report MTAD_E_CAPACITY early and the
 * attention launches carry blocks for keys that do not exist (harmless, slower). */
int mtad_seq_hint(mtad_ctx* ctx, int seq, int32_t kv_len);

/* Warp the target's distributions before the verification rule and the extra token, as in the paper's experiments
 * (App. F; the footnote to Sec. 3.2 states that the method is equally valid on warped distributions): every row of
 * P keeps its top_k most likely tokens, renormalised; of these, in descending order of probability (lower token id
 * first among equals), the first ones whose cumulative probability is larger than top_p are kept and renormalised,
 * the rest get probability 0.  A drafted token outside its row's kept set has probability 0 and cannot be accepted;
 * the extra token is drawn from the kept set.  The verify calls that follow then compute plain logits [rows, vocab]
 * into the workspace and derive the warped rows from them (row_lse of mtad_result is the log-sum-exp over the kept
 * tokens).  top_k = 0 switches warping off (the default); top_k <= 16 (MTAD_E_CAPACITY beyond), 0 < top_p <= 1
 * (MTAD_E_INVALID otherwise).  Host-side setting of the context, no launch.  The draft log-likelihoods passed to
 * the verify calls are the caller's; mtad_set_draft_warp (below) makes mtad_draft sample from warped rows too. */
int mtad_set_warp(mtad_ctx* ctx, int top_k, float top_p);

/* The same warping for the auxiliary model's rows in mtad_draft (App. F warps both models): every beam row
 * q(. | beam) keeps its top_k most likely tokens, renormalised, of these the first ones whose cumulative probability is
 * larger than top_p, renormalised again; the draft samples from these rows and reports their likelihoods (node_logq,
 * logq_ref).  A dropped token is never drafted.  When the rows of a step keep fewer (beam, token) pairs than
 * beam_width, the step keeps that many beams and the layer holds fewer nodes: node ids stay consecutive, n_nodes of
 * mtad_draft gives the count and becomes a required argument.  top_k = 0 switches it off (the default); limits and
 * errors as for mtad_set_warp; MTAD_E_INVALID without an auxiliary model.  Host-side setting, no launch. */
int mtad_set_draft_warp(mtad_ctx* ctx, int top_k, float top_p);

/* Draft with the auxiliary model: beam sampling of width beam_width for gamma steps (Sec. 2.1, the p_beam
 * equation; every intermediate beam becomes a tree node, Sec. 3.3).  At each step the beam_width kept sequences
 * are drawn without replacement, proportionally to their joint likelihood, as the beam_width largest values of
 * log q(beam) + log q(token | beam) + Gumbel noise, noise = -log(-log(u)).
 *   seqs        host  [B]                 sequence ids (distinct)
 *   keep_all_candidates  0: the tree holds the kept beams, W = beam_width nodes a layer, best first (the paper's
 *               tree).  Non-zero: a layer also records the candidates that the selection looked at and did not
 *               keep, as leaves: W = beam_width^2 nodes a layer - the beam_width^2 best perturbed tokens of the
 *               single beam of step 1, afterwards beam by beam (in the order of the previous layer's kept beams)
 *               its beam_width best perturbed tokens, best first.  The kept beams are the beam_width best of the
 *               layer; only they have children.  Needs gamma * beam_width^2 <= MTAD_MAX_NODES and a vocabulary of
 *               at least beam_width^2 tokens (MTAD_E_CAPACITY otherwise).
 *   uniforms    device [B, gamma, beam_width, vocab] fp32 in (0,1)
 *   n_nodes     device [B] int32, may be NULL   gamma * W, for the mtad_verify_tree call that follows
 *   tok,parent,depth  device [B, gamma * W] int32  node arrays, layer by layer (parent = -1: child of root)
 *   node_logq   device [B, gamma * W] fp32  joint draft log-likelihood of the path ending at each node
 *   logq_ref    device [B, gamma] fp32   log q(x**_{1:i}), x** = final beam with the highest likelihood
 *   best_path   device [B, gamma] int32  node ids of x**
 * The chain of Algorithm 1 is best_path with logq_ref.  kv_commit after a verification of this tree (or of that
 * chain) also rolls the auxiliary cache forward: accepted nodes that were beams of a layer before the last keep
 * their keys and values, an accepted node that the auxiliary model never ran (last layer, or a candidate that was
 * not kept) is replayed by the next draft together with the extra token. */
int mtad_draft(mtad_ctx* ctx, int B, const int32_t* seqs, int gamma, int beam_width, int keep_all_candidates,
               const float* uniforms, int32_t* n_nodes, int32_t* tok, int32_t* parent, int32_t* depth,
               float* node_logq, float* logq_ref, int32_t* best_path, void* stream);

/* Verify a draft chain x_1..x_gamma (Algorithm 1 from "P <- M_p(input, X)" to the return).
 *   seqs         host   [B]
 *   draft_tok    device [B, gamma] int32
 *   draft_logq   device [B, gamma] fp32, draft_logq[b,i] = log q(x_{1:i+1} | input) (joint)
 *   log_tau      log of the threshold tau in [0,1): <= 0, -INFINITY for tau = 0.  Prefix j passes iff
 *                log p(x_{1:j}) - log q(x_{1:j}) > log_tau (min(1, p/q) > tau, Sec. 3.2); the longest passing
 *                prefix is accepted, all gamma prefixes are tested.
 *   bonus_uniform device [B, vocab] fp32 in (0,1): the extra token is argmax_j(logit_j - log(-log u_j)), a draw
 *                from the target row after the accepted prefix. */
int mtad_verify_chain(mtad_ctx* ctx, int B, const int32_t* seqs, int gamma, const int32_t* draft_tok,
                      const float* draft_logq, float log_tau, const float* bonus_uniform,
                      const mtad_result* out, void* stream);

/* The rule of vanilla speculative decoding (Sec. 2.2, steps 2-4) on a draft chain, as a second accept mode on the
 * same target forward: token i is accepted iff accept_uniform[i] < min(1, p_i(x_i) / q_i(x_i)); the scan stops at
 * the first rejection, whose position is resampled from norm(max(0, p_i - q_i)); with every token accepted one more
 * token is drawn from the target's next row.  The last draw is a Gumbel-argmax over log of those weights with noise
 * from resample_uniform (lowest token id on ties).
 *   draft_tok        device [B, gamma] int32
 *   draft_logq_rows  device [B, gamma, vocab] fp32  the auxiliary model's normalised log-distribution at every
 *                    draft position (the whole row: the residual needs q at every token)
 *   accept_uniform   device [B, gamma] fp32 in (0,1);  resample_uniform  device [B, vocab] fp32 in (0,1)
 * Outputs as for mtad_verify_chain (path[i] = i; margin[0] = smallest |log u - log ratio| over the tested
 * positions); kv_commit follows as usual.  The verify forward computes plain logits [rows, vocab] into the
 * workspace; a warping set by mtad_set_warp is not applied in this mode.  gamma >= 1. */
int mtad_verify_chain_spd(mtad_ctx* ctx, int B, const int32_t* seqs, int gamma, const int32_t* draft_tok,
                          const float* draft_logq_rows, const float* accept_uniform, const float* resample_uniform,
                          const mtad_result* out, void* stream);

/* Verify a candidate tree (Sec. 3.3).  Node n of sequence b has token tok[b,n] and parent parent[b,n] (< n, or
 * -1 for a child of the root); n_nodes[b] <= max_nodes nodes are valid (n_nodes NULL: all max_nodes).
 * Candidate n at depth i passes iff log p(path to n) - logq_ref[b, i-1] > log_tau with
 * logq_ref[b, i-1] = log q(x**_{1:i}); the deepest passing node wins, ties by the larger target likelihood,
 * then by the lower index.
 *   n_nodes   device [B] int32;  tok, parent device [B, max_nodes] int32;  logq_ref device [B, max_depth] fp32 */
int mtad_verify_tree(mtad_ctx* ctx, int B, const int32_t* seqs, const int32_t* n_nodes, int max_nodes,
                     int max_depth, const int32_t* tok, const int32_t* parent, const float* logq_ref,
                     float log_tau, const float* bonus_uniform, const mtad_result* out, void* stream);

/* Keep the root row and the accepted path of the last verify call on this context (res = the same arrays, B and
 * seqs the same), drop every other draft row, advance L by eta + 1 and make the extra token the new root; the
 * auxiliary cache rolls forward the same way when the context has one and mtad_draft produced the tree.
 * Sequences whose status is non-zero are left untouched. */
int kv_commit(mtad_ctx* ctx, int B, const int32_t* seqs, const mtad_result* res, void* stream);

/* The paper has no counterpart for this entry point; it exists for callers that cannot allocate device memory.
 * Some hosts of this library - a plug-in running inside another engine's memory pool, a process whose CUDA
 * allocator has been frozen after start-up, code that may run while a stream is being captured - are not allowed
 * to call cudaMalloc, so they cannot supply the workspace that mtad_create wants.  This call verifies one draft
 * chain for ONE sequence exactly like mtad_verify_chain, but takes its scratch from a fixed array of
 * MTAD_STATIC_SCRATCH_BYTES that is compiled into the library (every GPU that loads the library holds that much
 * memory until the process exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   target      descriptor as for mtad_create; its kv_cache must be laid out for max_batch = 1
 *   kv_len      committed length of the sequence, root_token its last emitted token
 *   draft_tok, draft_logq, log_tau, bonus_uniform, out: as mtad_verify_chain with B = 1 (device arrays of the caller)
 * The K/V rows of the root and the draft tokens are left in cache slots kv_len .. kv_len + gamma, as after
 * mtad_verify_chain; there is no commit step, the caller keeps the rows it accepts.
 * Limits and sharing: returns MTAD_E_WORKSPACE when the model shape or gamma needs more scratch than the array
 * holds (mtad_workspace_bytes(target, NULL, 1, gamma) tells how much).  All calls on a device share the one array,
 * which still contains the previous call's data: the library re-zeroes the whole array whenever the model or gamma
 * changes (after synchronising the device, so that earlier calls still running on any stream are over) and the
 * split-K counters at the start of every call, but two calls whose GPU work overlaps (different streams, different threads) race
 * on it - issue them on one stream or synchronise in between.  The first call on a device (and any call that
 * changes the model or gamma) looks up the array's device address, zeroes it and synchronises the device; make
 * that call before starting a stream capture. */
#define MTAD_STATIC_SCRATCH_BYTES (16u << 20)
int mtad_verify_chain_static(const mtad_model_desc* target, int32_t kv_len, int32_t root_token, int gamma,
                             const int32_t* draft_tok, const float* draft_logq, float log_tau,
                             const float* bonus_uniform, const mtad_result* out, void* stream);

/* Instrumentation (not part of the method).  Kernel classes for mtad_profile_end. */
enum { MTAD_K_PREPARE = 0, MTAD_K_NORM, MTAD_K_GEMM, MTAD_K_ROPE, MTAD_K_ATTN, MTAD_K_LMRED, MTAD_K_ACCEPT,
       MTAD_K_COMMIT, MTAD_K_CLASSES };

/* Start bracketing every kernel launch of this context with a pair of CUDA events on the launching stream (room
 * for max_launches launches; later launches go unrecorded).  Creates events, no device memory. */
int mtad_profile_begin(mtad_ctx* ctx, int max_launches);
/* Grouped bracketing (call before mtad_profile_begin; on != 0): one event pair around every run of consecutive
 * launches of the same class instead of one per launch.  An event between two launches keeps the second from
 * starting before the first has drained, so per-launch brackets time every kernel as if it stood alone; a run's
 * bracket times its launches as they overlap in the real step.  MTAD_E_INVALID while profiling is on. */
int mtad_profile_grouped(mtad_ctx* ctx, int on);
/* Stop, synchronise the device and sum per kernel class: elapsed milliseconds, algorithmic bytes (bf16 weight
 * bytes of the GEMM launches; 0 for the other classes) and launch count.  Arrays of MTAD_K_CLASSES, host. */
int mtad_profile_end(mtad_ctx* ctx, double* ms, double* bytes, int64_t* launches);
/* Kernels of this library enqueued by this process so far. */
uint64_t mtad_kernel_launches(void);
/* Runs the weight-streaming tensor-core GEMM alone: y[T, N] (fp32, device) = x[T, K] (fp32, device) * W[N, K]^T
 * (bf16, device, 16-byte aligned), T <= 256, K a multiple of 8 and at most the context's largest FFN width.
 * variant 0: the stream-K kernel (work units dealt out evenly, partial tiles summed through the workspace);
 * variant 1: the cluster kernels (split-K inside a thread-block cluster, partial rows summed through distributed
 * shared memory; one kernel for up to 32 rows, one beyond) - MTAD_E_UNIMPLEMENTED where the shape does not suit them
 * (more than 256 accumulator columns, more tiles than co-resident CTAs).
 * For unit tests and kernel timing; uses the context's workspace. */
int mtad_debug_gemm(mtad_ctx* ctx, const void* W, int N, int K, const float* x, int T, float* y, int variant,
                    void* stream);

/* Extent audit (host arithmetic only: no device, no driver, descriptors may carry null pointers).  For one call on a
 * context created with (target, aux, max_batch, max_nodes) it lists, per array the call's kernels touch - every region
 * of the workspace, the KV caches, the caller's arrays - `reach`, one past the largest element index the kernels form
 * into it, and `extent`, the elements it holds; reach <= extent must hold everywhere.  call: MTAD_AUDIT_VERIFY (B
 * sequences of nodes + 1 rows, depth gamma), MTAD_AUDIT_DRAFT (mtad_draft with gamma, beam; every step), or
 * MTAD_AUDIT_COMMIT (kv_commit after such a verify).  len_ub: largest committed length of the sequences.  Writes at
 * most max_out records, *n_out = records there are; `what` points at static strings. */
typedef struct mtad_extent { const char* what; int64_t reach; int64_t extent; } mtad_extent;
enum { MTAD_AUDIT_VERIFY = 0, MTAD_AUDIT_DRAFT = 1, MTAD_AUDIT_COMMIT = 2 };
int mtad_audit_extents(const mtad_model_desc* target, const mtad_model_desc* aux, int max_batch, int max_nodes,
                       int call, int B, int nodes, int gamma, int beam, int64_t len_ub, mtad_extent* out,
                       int max_out, int* n_out);

/* Every array of the workspace is followed by 64 guard bytes written at mtad_create.  Synchronises the stream, reads
 * them back and returns how many arrays have damaged guards (0: none; *damaged, if given, names the first one) - a
 * write past the end of a workspace array that happened to land in mapped memory shows up here.  For tests. */
int mtad_debug_check_canaries(mtad_ctx* ctx, void* stream, const char** damaged);

/* Where the workspace array `name` (the names the extent audit reports) lies: byte offset from the workspace base,
 * element count and element size.  For tests that inspect intermediate results. */
int mtad_debug_region(const mtad_ctx* ctx, const char* name, size_t* offset, size_t* count, size_t* elem_bytes);

/* Test hook for the time-out path: wait_limit = iterations a bounded wait inside the GEMM kernels may poll (0: the
 * default); no_operands != 0 makes the GEMM kernels leave out their operand-row copies, so the waits on them run out
 * and every sequence of the call reports MTAD_ST_TIMEOUT.  The kernels return normally; a later call with the hook
 * switched off is unaffected. */
int mtad_debug_set_wait(mtad_ctx* ctx, unsigned int wait_limit, int no_operands);

const char* mtad_status_str(int status);
int mtad_last_cuda_error(const mtad_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MTAD_H_ */
