/* hivis.h - C ABI of the HiViS drafter step on one NVIDIA B200 (sm_100a).
 *
 * The library runs the drafter side of HiViS speculative decoding: a single
 * Llama-style decoder layer that never sees visual tokens.  Its input at each
 * text position is an FC (2d -> d) fusion of the target VLM's hidden state
 * with the embedding of the following token, plus a step-indexed
 * bias-correction residual; its KV cache holds text positions only.
 *
 * Conventions shared by every call
 *   - Every pointer is a DEVICE pointer unless its name ends in `_host`.
 *   - Device pointers must be 16-byte aligned.
 *   - All matrices are row-major [out, in]:  y = W x.
 *   - The caller owns every buffer it passes.  hivis_init copies the weights
 *     into library-owned memory (the caller may free its copies once the
 *     stream has finished); hivis_destroy frees everything the library owns.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, 0 = the
 *     default stream) and return without waiting; outputs are valid once the
 *     stream has been synchronised.  A context must always be used with work
 *     ordered on one stream at a time, and is not thread-safe.
 *   - Every function returns HIVIS_OK (0) or a negative error code and never
 *     throws.  After an error nothing was launched unless the code is
 *     HIVIS_ERR_CUDA.  hivis_last_error gives a text for the last failure.
 *   - A sequence lives in a `slot` in [0, max_batch).  Batched calls take the
 *     slots they work on in `seq_slots_host` (B ints, all different); NULL
 *     means slots 0..B-1.
 */
#ifndef HIVIS_H
#define HIVIS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hivis_ctx hivis_ctx;

enum {
    HIVIS_OK = 0,
    HIVIS_ERR_ARG = -1,      /* null / misaligned pointer, bad scalar argument            */
    HIVIS_ERR_SHAPE = -2,    /* dimensions the kernels do not support                     */
    HIVIS_ERR_DTYPE = -3,    /* unknown element type                                      */
    HIVIS_ERR_STATE = -4,    /* call out of order (draft without a pending pair, ...)     */
    HIVIS_ERR_CAPACITY = -5, /* would exceed max_batch / max_len / max_k                  */
    HIVIS_ERR_CUDA = -6,     /* a CUDA runtime call failed                                */
    HIVIS_ERR_TIMEOUT = -7,  /* a bounded device-side wait ran out                        */
    HIVIS_ERR_NOMEM = -8     /* device or host allocation failed                          */
};

enum { HIVIS_F32 = 0, HIVIS_BF16 = 1 };

#define HIVIS_MAX_BATCH 64   /* upper limit for hivis_config.max_batch */
#define HIVIS_MAX_K 16       /* upper limit for hivis_config.max_k     */

typedef struct {
    uint32_t struct_size;    /* sizeof(hivis_config), checked                              */
    int dtype;               /* HIVIS_F32 | HIVIS_BF16: weights, hidden states, residual   */
                             /* rows and the KV cache are all stored in this type          */
    int d;                   /* model width; multiple of 8                                 */
    int n_q_heads, n_kv_heads;   /* n_q_heads % n_kv_heads == 0                            */
    int head_dim;            /* 64 or 128                                                  */
    int ffn;                 /* SwiGLU inner width; multiple of 8                          */
    int vocab;
    float rms_eps;
    float rope_base;
    int max_batch;           /* number of sequence slots, 1..HIVIS_MAX_BATCH               */
    int max_len;             /* KV rows per slot                                           */
    int max_k;               /* longest draft chain, 1..HIVIS_MAX_K                        */
} hivis_config;

/* The drafter's parameters (paper Sec. 3.2 and Algorithm 1).  `embed` and `lm_head` are the
 * target model's own tables, which the drafter reuses.  `fc` is the semantic-fusion layer:
 * columns [0,d) multiply the hidden feature (the paper's w1, stored transposed), columns
 * [d,2d) the token embedding (w2).  `resid_proj` is the paper's w that projects a residual
 * row r^i (rho_i = resid_proj * r_i); NULL means the rows passed to prefill/draft are used
 * as given.  bq/bk/bv are optional QKV biases.                                              */
typedef struct {
    const void* embed;      /* [vocab, d]                    */
    const void* lm_head;    /* [vocab, d]                    */
    const void* fc;         /* [d, 2d]                       */
    const void* norm1;      /* [d]  RMSNorm gain before QKV  */
    const void* wq;         /* [n_q_heads*head_dim, d]       */
    const void* wk;         /* [n_kv_heads*head_dim, d]      */
    const void* wv;         /* [n_kv_heads*head_dim, d]      */
    const void* bq;         /* nullable                      */
    const void* bk;         /* nullable                      */
    const void* bv;         /* nullable                      */
    const void* wo;         /* [d, n_q_heads*head_dim]       */
    const void* norm2;      /* [d]  RMSNorm gain before MLP  */
    const void* w_gate;     /* [ffn, d]                      */
    const void* w_up;       /* [ffn, d]                      */
    const void* w_down;     /* [d, ffn]                      */
    const void* resid_proj; /* [d, d], nullable              */
} hivis_weights;

/* Create a context on the current CUDA device: validates the configuration, copies (and
 * re-lays-out) the weights, allocates the text-only KV cache [max_batch][n_kv_heads][max_len]
 * [head_dim] x2 and all workspaces.  The only call that allocates device memory.
 * Errors: ARG (null, misaligned, struct_size), SHAPE, DTYPE, CAPACITY, NOMEM, CUDA.          */
int hivis_init(hivis_ctx** out, const hivis_config* cfg, const hivis_weights* w, void* stream);

/* Waits for the device to finish and frees everything the context owns.  NULL is allowed.   */
int hivis_destroy(hivis_ctx* ctx);

/* Prefix build (Algorithm 1, the prefix build; Eq. 1).  Appends text positions to B sequences.
 * The batch is packed: sequence b owns entries [cu_seqlens_host[b], cu_seqlens_host[b+1]) of
 * `ids` (int32) and of `hidden` ([total, d], ctx dtype), T_b >= 1 entries each.  Entry p is
 * the pair (target hidden state of text token p, id of text token p+1): the causal shift of
 * Sec. 3.2 is already applied by the caller.  For every pair but the last of each sequence
 * the library computes fuse -> +rho_0 -> RMSNorm -> K,V projections -> RoPE(K) and stores the
 * K/V rows (with one decoder layer nothing else of a prefix position is ever read).  The last
 * pair of each sequence is kept as the PENDING pair that draft step 0 consumes.
 * start_pos_host: NULL appends after the rows the slot holds now; otherwise start_pos_host[b]
 * (0 <= start <= current length) first truncates the slot to that many rows, which lets the
 * caller overwrite rows that came from drafting by rows built from true target features.
 * A slot whose pending pair has not been drafted yet cannot be appended to (STATE): the row
 * of that pair was never cached, so the new rows would land one position too early.  Pass the
 * whole continuation in one call, or pass start_pos and repeat the pair.
 * resid0: [d] in ctx dtype = the initial residual r^0 (projected by resid_proj when the
 * context has one); NULL = no residual.
 * Errors: ARG, STATE, CAPACITY (rows + T_b - 1 + max... > max_len), CUDA.                    */
int hivis_prefill(hivis_ctx* ctx, int B, const int* seq_slots_host, const int32_t* ids,
                  const void* hidden, const int32_t* cu_seqlens_host,
                  const int32_t* start_pos_host, const void* resid0, void* stream);

/* k chained greedy draft steps for B sequences (Algorithm 1, the drafting loop; Eq. 2).  Step 0 runs
 * the pending pair at the next cache row; step s >= 1 runs (the layer output of step s-1, the
 * token chosen at step s-1).  Each step: fuse + residual row min(s, n_resid-1) (rows beyond
 * the trained ones reuse the last, "Training Setup"), RMSNorm, QKV, RoPE, causal attention
 * over the slot's cache, O projection, SwiGLU MLP, LM head, argmax (lowest index on ties).
 * Every step appends one K/V row, so the slot grows by k rows.
 * resid: [n_resid, d] in ctx dtype (projected by resid_proj when present); NULL = none.
 * out_ids: int32 [B, k].
 * forced_ids (nullable, int32 [B, k]): teacher forcing for parity tests - the token fed to
 * step s+1 is forced_ids[b, s]; out_ids still reports each step's own argmax.
 * out_logits (nullable, fp32 [B, k, vocab]): every step's LM-head output.
 * Errors: ARG, STATE (a listed slot has no pending pair), CAPACITY (k > max_k or the slot
 * would exceed max_len), CUDA.                                                                */
int hivis_draft(hivis_ctx* ctx, int B, const int* seq_slots_host, int k, const void* resid,
                int n_resid, int32_t* out_ids, const int32_t* forced_ids, float* out_logits,
                void* stream);

/* The same k chained draft steps with every step's token DRAWN from softmax(logits / temperature)
 * instead of taken as the maximum (the paper also evaluates T = 1, "Inference Setup").  The
 * draw is the Gumbel-max rule: token = argmax_i (logits_i / T - log(-log u_i)), lowest index
 * among equal values, which turns one uniform number per vocabulary entry into an exact sample
 * of that distribution; the uniform numbers are the caller's.
 * uniforms: fp32 [B, k, vocab], device, every value in (0, 1).
 * out_logits (nullable, fp32 [B, k, vocab]): the unperturbed LM-head outputs - the drafter's
 * distributions that hivis_verify_sampled needs.
 * Runs in the chain kernels only: one sequence, or up to 16 sequences of a bf16 context;
 * anything else returns SHAPE.  Otherwise as hivis_draft (state, growth of the slots, errors;
 * ARG also for temperature <= 0).                                                             */
int hivis_draft_sampled(hivis_ctx* ctx, int B, const int* seq_slots_host, int k, const void* resid,
                        int n_resid, float temperature, const float* uniforms, int32_t* out_ids,
                        float* out_logits, void* stream);

/* Batched greedy verification and KV rollback (Sec. 2.1; Algorithm 1, the verification step).
 * target_logits: [B, k+1, vocab] in logits_dtype (HIVIS_F32 | HIVIS_BF16); row j is the
 * target's prediction after the root token and j draft tokens.  Draft token j (0-based) is
 * accepted iff it equals argmax(row j) (lowest index on ties) and all earlier ones were.
 * out_accept[b] = n in [0, k]; out_next[b] = argmax(row n) (correction or bonus token);
 * the slot is rolled back to (rows before the draft) + 1 + min(n, k-1) rows, also written to
 * out_kv_len[b] (nullable).  The pending pair is consumed.  Must follow a hivis_draft of the
 * same k on the same slots.
 * Errors: ARG, DTYPE, STATE, CUDA.                                                            */
int hivis_verify(hivis_ctx* ctx, int B, const int* seq_slots_host, int k,
                 const int32_t* draft_ids, const void* target_logits, int logits_dtype,
                 int32_t* out_accept, int32_t* out_next, int32_t* out_kv_len, void* stream);

/* Verification by speculative sampling, for drafts whose tokens were DRAWN from the drafter's distribution
 * (Sec. 2.1: the target keeps the drafted tokens that are consistent with its distribution, drops the first
 * that is not together with all that follow and re-draws the next token accordingly; the rule is the one of
 * Leviathan et al. and Chen et al., which the section cites).  With p_j = softmax(target row j / T) and
 * q_j = softmax(drafter row j / T): draft token j is kept while u_accept[b, j] < min(1, p_j(x) / q_j(x));
 * n = number kept; the next token is drawn by inverse CDF at u_sample[b] from max(0, p_n - q_n) (n < k) or
 * from p_k (n = k): the first token whose cumulative mass exceeds u_sample[b] times the total mass.
 *   draft_logits fp32 [B, k, vocab]: the drafter's logits of the k steps (out_logits of hivis_draft_sampled / hivis_draft);
 *   target_logits [B, k+1, vocab] in logits_dtype; temperature > 0;
 *   u_accept fp32 [B, k], u_sample fp32 [B]: uniform numbers in [0, 1) supplied by the caller;
 *   outputs and rollback as for hivis_verify.  Must follow a draft call of the same k on the same slots.
 * Errors: ARG, DTYPE, STATE, CAPACITY, CUDA.                                                            */
int hivis_verify_sampled(hivis_ctx* ctx, int B, const int* seq_slots_host, int k, const int32_t* draft_ids,
                         const float* draft_logits, const void* target_logits, int logits_dtype,
                         float temperature, const float* u_accept, const float* u_sample,
                         int32_t* out_accept, int32_t* out_next, int32_t* out_kv_len, void* stream);

/* Tree drafting for ONE sequence (Sec. 2.1: the paper drafts with the dynamic draft tree of EAGLE-2;
 * "Inference Setup": top-10 expansion, depth 6, the 60 paths of highest cumulative probability kept;
 * supplementary material, Sec. A: 8 per expansion, depth 4, 30 kept).
 * Level 0 runs the slot's pending pair at its next cache row P and proposes the `topk` most probable
 * tokens.  Level l = 1..depth-1 runs the `topk` candidates of depth l with the highest cumulative
 * log-probability (the frontier) as one batch: input = (layer output of the forward that proposed the
 * node, the node's token) at position P + l, residual row min(l, n_resid-1), attention over the prefix,
 * the node's ancestors and itself; each proposes `topk` candidates of depth l + 1, score = parent's score
 * + log-softmax(logits)[token].  Of all topk + (depth-1)*topk^2 candidates the `keep` with the highest
 * score are returned in creation order (level by level, parents in frontier order, children by rank), so
 * a node's parent precedes it.  Equal scores: the candidate created first; equal logits: the lower token.
 *   out_tokens, out_parents (index into the list, -1 = child of the root) int32 [keep], out_scores fp32
 *   [keep], out_count int32 [1] = number of nodes written (min(keep, number of candidates)).
 * The slot's row count does not change until hivis_verify_tree; rows [P, P + 1 + (depth-1)*topk) of the
 * slot are used for the tree's K/V rows, so that many rows must be free (CAPACITY otherwise).
 * Limits: 1 <= topk <= HIVIS_TREE_MAX_TOPK, 1 <= depth <= max_k, 1 <= keep <= HIVIS_TREE_MAX_KEEP.
 * Errors: ARG, STATE (no pending pair), CAPACITY, CUDA.                                              */
#define HIVIS_TREE_MAX_TOPK 16
#define HIVIS_TREE_MAX_KEEP 256
int hivis_draft_tree(hivis_ctx* ctx, int slot, int topk, int depth, int keep, const void* resid, int n_resid,
                     int32_t* out_tokens, int32_t* out_parents, float* out_scores, int32_t* out_count,
                     void* stream);

/* Greedy verification of the tree drafted last on the slot, and KV compaction (Sec. 2.1; Algorithm 1,
 * the verification step).  target_logits: [count + 1, vocab] in logits_dtype: row 0 is the target's prediction after
 * the root token, row 1 + i its prediction after the path that ends in kept node i.  From the root, the
 * child that carries argmax(row of the current node) is accepted (lowest index on ties) for as long as
 * there is one.  out_accept[0] = n accepted nodes (0..depth), out_path int32 [depth] = their indices
 * (-1 beyond n), out_next[0] = argmax(row of the last accepted node): the correction or bonus token.
 * The slot then holds P + 1 + m rows (also written to out_kv_len, nullable): the root's row and, right
 * behind it in path order, the K/V rows of the m accepted nodes that were run through the layer (nodes
 * of the last level were not, like the last token of a chained draft).  Must follow hivis_draft_tree on
 * the slot.  Errors: ARG, DTYPE, STATE, CUDA.                                                        */
int hivis_verify_tree(hivis_ctx* ctx, int slot, const void* target_logits, int logits_dtype,
                      int32_t* out_accept, int32_t* out_path, int32_t* out_next, int32_t* out_kv_len,
                      void* stream);

/* Forget a sequence: zero rows, no pending pair.                                              */
int hivis_reset(hivis_ctx* ctx, int slot, void* stream);

/* Synchronises `stream` and reports the slot's row count and whether a pending pair exists.  */
int hivis_get_kv_len(hivis_ctx* ctx, int slot, int* n_rows_host, int* pending_host, void* stream);

/* Set the slot's row count (0 <= n_rows <= max_len) without touching the cached data; with
 * restore_pending != 0 the pair stored by the last prefill becomes pending again.  Lets a
 * benchmark return to the state right after prefill between timed repetitions.               */
int hivis_set_kv_len(hivis_ctx* ctx, int slot, int n_rows, int restore_pending, void* stream);

/* The same for B slots in one launch: slots_host[b] (NULL = slots 0..B-1, each at most once) gets
 * n_rows_host[b] rows.  Errors: ARG, STATE, CAPACITY as above; nothing is changed when one is returned. */
int hivis_set_kv_len_batch(hivis_ctx* ctx, int B, const int* slots_host, const int* n_rows_host,
                           int restore_pending, void* stream);

/* Debug: copy rows [row0, row0+n) of the slot's K and V cache, widened to fp32, into
 * out_k / out_v, each [n, n_kv_heads*head_dim].                                               */
int hivis_read_kv(hivis_ctx* ctx, int slot, int row0, int n, float* out_k, float* out_v,
                  void* stream);

/* Debug: copy an intermediate of the LAST draft step of the last hivis_draft call, fp32,
 * [B, width] in call order: U fused input (d), ATTN attention output (n_q_heads*head_dim),
 * Y post-attention residual (d), ACT SwiGLU product (ffn), G layer output (d), Q the query
 * projection with its bias and BEFORE the rotary embedding (n_q_heads*head_dim).  The K and V
 * rows of that step are the slot's newest cache rows: read them with hivis_read_kv (K after
 * the rotary embedding, as stored).                                                          */
enum { HIVIS_TAP_U = 0, HIVIS_TAP_ATTN = 1, HIVIS_TAP_Y = 2, HIVIS_TAP_ACT = 3, HIVIS_TAP_G = 4, HIVIS_TAP_Q = 5 };
int hivis_debug_tap(hivis_ctx* ctx, int which, float* out, void* stream);

/* Options.
 * HIVIS_OPT_CHAIN_KERNEL (default 1): a draft of ONE sequence runs all k steps in a single persistent
 * cooperative kernel of fp32 FMAs (one CTA per SM, grid barriers between the phases of a step, weights
 * prefetched across them by per-warp bulk-copy rings).
 * HIVIS_OPT_TC_KERNEL (default 1): with bf16 weights and d a multiple of 64, a draft of 2..16 sequences
 * runs all k steps in one persistent cooperative kernel that streams the weights with TMA and multiplies
 * on the tcgen05 tensor cores (weights as the M operand, batch as N); 2 = use it for one sequence as well;
 * 0 = never.  What neither kernel takes runs as separate kernel launches per step.  All paths give the
 * same results up to fp32 summation order and the bf16 rounding of the tensor-core operand.
 * HIVIS_OPT_WAIT_LIMIT_US (default 1 000 000): how long a device-side wait of the chain kernels (grid
 * barrier, copy completion) may last before the kernel gives up, raises the error word that hivis_status
 * reports and returns in an orderly way.
 * HIVIS_OPT_DEBUG_MISS_BARRIER (test aid): 1 makes the grid barriers of the NEXT hivis_draft call
 * impossible to complete, so that every wait runs into its limit: hivis_status then returns
 * HIVIS_ERR_TIMEOUT and the context is usable again.  Nothing faults or hangs.
 * HIVIS_OPT_PHASE_TIMES (default 0): 1 makes the tensor-core chain kernel write a time stamp per CTA at the
 * events listed under hivis_read_phase_times (a store per event; off, the kernel only tests a pointer).
 * HIVIS_OPT_L2_KEEP (default 0): bit mask over the six weight matrices of a step (bit 0 fusion FC, 1 QKV, 2 O,
 * 3 gate/up, 4 down, 5 LM head).  The tensor-core chain kernel loads the weights of the named matrices with the
 * keep-in-L2 policy instead of streaming them through: with k chained steps in one launch a subset that fits
 * in L2 beside the KV cache is then read from HBM once per launch rather than once per step.
 * HIVIS_OPT_TC_PREFILL (default 1): with bf16 weights, a hivis_prefill call of HIVIS_TC_PREFILL_MIN_PAIRS pairs or more
 * builds the prefix with two tcgen05 GEMMs over all pairs at once (weights as the M operand, 128 pairs as N); 0 = always
 * the 16-pairs-per-pass kernels, which smaller calls use in any case; a value n > 1 = calls of n pairs or more.
 * Same results up to fp32 summation order.                                                                     */
#define HIVIS_TC_PREFILL_MIN_PAIRS 17     /* more than one pass of the 16-pairs kernels: measured crossover */
enum { HIVIS_OPT_CHAIN_KERNEL = 0, HIVIS_OPT_TC_KERNEL = 1, HIVIS_OPT_WAIT_LIMIT_US = 2, HIVIS_OPT_DEBUG_MISS_BARRIER = 3,
       HIVIS_OPT_PHASE_TIMES = 4, HIVIS_OPT_L2_KEEP = 5, HIVIS_OPT_TC_PREFILL = 6 };
int hivis_set_option(hivis_ctx* ctx, int option, int value);

/* Where the time of a draft step goes: synchronises `stream` and copies the time stamps of the LAST hivis_draft
 * that ran the tensor-core chain kernel with HIVIS_OPT_PHASE_TIMES on.  out_host[(s * HIVIS_PHASE_EVENTS + e) *
 * grid + cta] = time in ns (the GPU's global timer) of event e of draft step s on CTA cta; 0 where the event did
 * not occur (a CTA without work in a phase).  Events:
 *   0..7   the CTA's arrival on the grid barrier after: embedding gather, fusion FC, QKV, attention, O, gate/up,
 *          down, LM head (the time from the last arrival on one barrier to the last arrival on the next is what
 *          that phase costs);
 *   8..13  the CTA's operand producer got past its wait for the phase's input (FC, QKV, O, gate/up, down, LM head);
 *   14..19 the last accumulator of the CTA's range in that phase was complete (what follows is the phase's tail:
 *          partial sums, output stage, barrier);
 *   20     the CTA's attention warps got past their wait for the QKV phase.
 * k_host, grid_host: draft steps and CTAs recorded.  capacity: entries out_host can take; with less than
 * k * HIVIS_PHASE_EVENTS * grid the call fills k_host and grid_host and returns HIVIS_ERR_CAPACITY.
 * Errors: ARG, STATE (nothing recorded), CAPACITY, CUDA.                                                    */
#define HIVIS_PHASE_EVENTS 24
int hivis_read_phase_times(hivis_ctx* ctx, uint64_t* out_host, long long capacity, int* k_host, int* grid_host,
                           void* stream);

/* Synchronises `stream` and reports what the kernels since the last call recorded:
 * HIVIS_ERR_TIMEOUT - a kernel gave up on a bounded device-side wait (the outputs of that call
 *   are invalid, the context stays usable);
 * HIVIS_ERR_ARG - a token id outside [0, vocab) reached the embedding lookup (ids passed to
 *   hivis_prefill, forced_ids of hivis_draft; they live in device memory, so the host cannot
 *   check them): the kernels read it as token 0 and went on, nothing faulted.
 * Otherwise HIVIS_OK.  The record is cleared by the call.                                       */
int hivis_status(hivis_ctx* ctx, void* stream);

/* Per-kernel timing of hivis_draft.  Between hivis_profile_begin and hivis_profile_end every
 * kernel the draft chain launches is bracketed by CUDA events on its stream (this slows the chain
 * slightly, so time whole chains without it).  hivis_profile_end waits for the last event and adds
 * up, per kernel class, the device time in ms and the number of launches; both arrays are host
 * arrays of HIVIS_PROFILE_CLASSES entries, indexed: 0 fuse FC, 1 QKV, 2 attention, 3 O projection,
 * 4 gate/up, 5 down, 6 LM head + argmax, 7 set-up and finish kernels, 8 the persistent chain
 * kernel (all k steps of one sequence in one launch).                                          */
#define HIVIS_PROFILE_CLASSES 9
int hivis_profile_begin(hivis_ctx* ctx);
int hivis_profile_end(hivis_ctx* ctx, float* ms_host, int64_t* launches_host);

/* Bytes of weights and KV that one draft step of the given batch must read at least once
 * (the roofline's numerator): weights once per step regardless of B, plus K and V rows
 * [0, rows_b] of every listed slot.  kv_rows_host[b] = rows the slot holds at that step.      */
int64_t hivis_step_bytes(const hivis_ctx* ctx, int B, const int* kv_rows_host);

/* Number of kernel launches the library has enqueued since the context was created.          */
int64_t hivis_launch_count(const hivis_ctx* ctx);

const char* hivis_last_error(const hivis_ctx* ctx);

/* Greedy verification that allocates nothing and needs no context.  (The paper has no counterpart:
 * this is the arithmetic of hivis_verify offered to callers that cannot obtain device memory, such
 * as a plug-in inside a server whose memory pool already owns the GPU, or code that runs after its
 * host has closed the allocation phase.)  The per-row argmax keys live in a fixed array inside the
 * library image, HIVIS_MAX_BATCH * (HIVIS_MAX_K + 1) 8-byte entries (8.5 KB) on every GPU that
 * loads the library, held until the process exits.  The call uses no cudaMalloc, cudaFree or other
 * allocating routine.
 *   draft_ids [B, k] int32, target_logits [B, k+1, vocab] in logits_dtype: as for hivis_verify.
 *   rows_before (nullable, int32 [B]): cache rows each sequence held before its draft; when given,
 *   out_kv_len[b] = rows_before[b] + 1 + min(n, k-1), the row count hivis_verify would roll the
 *   slot back to.  rows_before and out_kv_len are given together or both NULL.
 *   out_accept, out_next: as for hivis_verify.  No library state is read or changed.
 * The first call made with a given device current looks up the array's address on that device;
 * make that first call outside any stream capture.  All calls on one device share the array and
 * it keeps the previous call's contents (each call clears the part it uses on `stream` first), so
 * two calls whose work overlaps on the GPU, e.g. on different streams, race: order them.
 * Errors: CAPACITY (B > HIVIS_MAX_BATCH or k > HIVIS_MAX_K: the fixed array is too small), SHAPE,
 * DTYPE, ARG, CUDA; the text is available from hivis_last_error(NULL).                           */
int hivis_verify_noalloc(int B, int k, int vocab, const int32_t* draft_ids, const void* target_logits,
                         int logits_dtype, const int32_t* rows_before, int32_t* out_accept,
                         int32_t* out_next, int32_t* out_kv_len, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HIVIS_H */
