/* cod.h — C ABI of the Carryover drafting round for NVIDIA B200 (sm_100a).
 *
 * One "round" is what a block-diffusion drafter does between two target
 * verifications (paper: Section 2 "Carryover Drafting", Eq. 1-2; Appendix A,
 * Algorithm 1 and its "Cache semantics" paragraph):
 *
 *   1. greedy verify-accept of the drafted block against the target's tokens;
 *   2. projection of the target's concatenated multi-layer hidden states into
 *      drafter K/V through the existing fusion map F and the per-layer K_l, V_l,
 *      with the learned embedding E_carry added to the REJECTED rows only;
 *   3. accepted rows are appended to the paged committed drafter cache C_l,
 *      rejected rows replace the one-block carryover slot U_l;
 *   4. the next block ([bonus, MASK, ...]) attends to [C_l; U_l; block];
 *   5. the tied LM head with a fused argmax gives the next proposals.
 *
 * Beyond that default round: the complete drafter layer (cod_config.d_ff,
 * COD_F_QK_NORM), the round at temperature 1 (cod_verify_accept_stochastic,
 * cod_lm_head_sample, cod_draft_round_stochastic), the two other ways of
 * marking rejected rows the paper compares (COD_F_NO_CARRY_EMBED,
 * COD_F_REJ_PROJECTOR), retention of rejected rows over several rounds
 * (cod_config.carry_rounds) and three analysis aids (cod_taps.carry_mass,
 * cod_reconvergence_count, cod_lm_head_rank).
 *
 * Conventions
 *   - Every function returns 0 (COD_OK) or a negative cod_status. Nothing throws.
 *   - "device" pointers are CUDA device addresses owned by the caller and only
 *     borrowed for the call; "host" pointers are ordinary host addresses.
 *   - All work is enqueued on the caller's stream (a cudaStream_t passed as
 *     void*); no call synchronises the host except cod_create, cod_destroy
 *     and cod_poll_status. Results are valid once the stream has been
 *     synchronised by the caller. For small rounds cod_draft_round also uses a
 *     second stream owned by the context, forked from and joined back into the
 *     caller's stream with events (under stream capture these become graph
 *     edges); a context therefore serves one round at a time.
 *   - After cod_create the library allocates nothing (the workspace is sized
 *     from cod_config at creation).
 *   - What only the device can see (a position beyond the page table, a token
 *     id outside the vocabulary, an expired bounded wait) sets a bit in a sticky
 *     device status word; the offending access is skipped and the kernel ends
 *     normally. cod_poll_status copies the word out.
 *   - Element type: COD_BF16 = bfloat16 storage, COD_F32 = float storage, for
 *     weights, H, the KV pool, the carry slot, J, q/k/v/out. Accumulation,
 *     norms, softmax and the residual stream are float in both.
 *   - Layouts are row-major with the last index contiguous.
 */
#ifndef COD_H_
#define COD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cod_ctx cod_ctx;
typedef void* cod_stream_t; /* a cudaStream_t */

enum cod_status {
  COD_OK = 0,
  COD_ERR_INVALID_ARG = -1, /* NULL pointer, size out of range, misaligned pointer */
  COD_ERR_UNSUPPORTED = -2, /* a shape or flag this build has no kernel for */
  COD_ERR_CUDA = -3,        /* a CUDA runtime call or launch failed */
  COD_ERR_NO_WEIGHTS = -4,  /* cod_set_weights has not been called */
  COD_ERR_ALLOC = -5,       /* cod_create could not allocate its workspace */
  COD_ERR_TOO_LARGE = -6    /* a size exceeds a fixed capacity (see cod_lm_head_argmax_static) */
};

enum cod_dtype { COD_F32 = 0, COD_BF16 = 1 };
enum cod_mode {
  COD_CARRY = 0,   /* Algorithm 1, right column: all rows projected, rejected rows carried */
  COD_BASELINE = 1 /* Algorithm 1, left column: accepted rows only, U_l left empty */
};

/* cod_config.flags */
#define COD_F_HIDDEN_NORM 1u /* RMS-normalise (with gain g_hidden) the output of F */
#define COD_F_NO_TENSOR_CORES 2u /* use the plain-FMA kernels only (an on-GPU cross-check) */
/* Attention grids several waves deep run either as one CTA per (sequence, head, part) or as persistent CTAs that
   walk the longest-first work list without draining their pipelines between items. Same results either way; the
   library picks by geometry (persistent for 128 query rows per head group, i.e. block 32). These two force it: */
#define COD_F_ATTN_ONE_ITEM_CTAS 32u
#define COD_F_ATTN_PERSISTENT 64u
#define COD_F_NO_CARRY_EMBED 8u /* rejected rows pass F unmarked ("no explicit discrimination", Section 5) */
#define COD_F_REJ_PROJECTOR 16u /* rejected rows pass their own fusion map fc_rej instead of F + E_carry
                                   ("separate projector", Section 5; its shape is taken as F's) */
#define COD_F_QK_NORM 4u /* per-head RMS norm with gain (g_qnorm, g_knorm) of queries and of all keys,
                            cached and block keys alike, before the rotation */

/* bits of the sticky device status word */
#define COD_DEV_BAD_TOKEN 1u      /* a token id outside [0, vocab) was met (treated as id 0) */
#define COD_DEV_PAGE_OVERFLOW 2u  /* a position fell beyond max_pages_per_seq (row not stored) */
#define COD_DEV_BAD_PAGE 4u       /* block_table held a page id outside [0, n_pages) */
#define COD_DEV_TIMEOUT 8u        /* a bounded device-side wait gave up */
#define COD_DEV_BAD_LEN 16u       /* committed_len / carry_len outside its range */

/* Immutable description of the drafter and of the capacities the workspace is sized for. */
typedef struct {
  int32_t d_target;          /* width of one captured target layer                         */
  int32_t n_cap;             /* captured target layers; D_in = d_target * n_cap            */
  int32_t d_model;           /* drafter width D; must equal n_q_heads * head_dim           */
  int32_t n_layers;          /* drafter layers Ld                                          */
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t vocab;             /* LM head = transposed embedding table                       */
  int32_t mask_token_id;
  int32_t block;             /* W: rows of the verified window = drafted block size        */
  int32_t page_size;         /* tokens per KV page                                         */
  int32_t max_batch;         /* largest S any call will pass                               */
  int32_t max_pages_per_seq; /* row length of block_table                                  */
  int32_t n_pages;           /* pages in kv_pool (per layer)                               */
  int32_t dtype;             /* cod_dtype                                                  */
  uint32_t flags;
  float rope_theta, rms_eps;
  int32_t attn_split_len;    /* keys per attention split (a multiple of 32); 0 = library default */
  int32_t d_ff;              /* width of the gated MLP that follows the attention sub-layer of every
                                drafter layer (a multiple of 64); 0 = no MLP. The paper leaves the
                                drafter body open (Section 2.1); this is the complete-layer reading  */
  int32_t carry_rounds;      /* k: rounds for which rejected rows stay in the carry slot (0 or 1: the paper's
                                one-round slot; k > 1: U_l = the rejected rows of the last k rounds, oldest
                                first - the retention beyond a single round that Section 6 leaves open)   */
} cod_config;

/* Borrowed device pointers, element type per cod_config.dtype, each matrix [out, in]. */
typedef struct {
  const void* fc;       /* [D, D_in]            the fusion map F                           */
  const void* e_carry;  /* [D_in]               E_carry (Eq. 2)                            */
  const void* g_hidden; /* [D]                  gain of the norm after F                   */
  const void* wk;       /* [Ld][n_kv*hd, D]     K_l                                        */
  const void* wv;       /* [Ld][n_kv*hd, D]     V_l                                        */
  const void* wq;       /* [Ld][n_q*hd, D]                                                 */
  const void* wo;       /* [Ld][D, n_q*hd]                                                 */
  const void* g_attn;   /* [Ld][D]              gain of the pre-attention norm             */
  const void* g_final;  /* [D]                  gain of the final norm                     */
  const void* emb;      /* [vocab, D]           embedding table = LM head                  */
  /* complete layer only; may be NULL when d_ff == 0 resp. COD_F_QK_NORM is not set:               */
  const void* w_gate;   /* [Ld][d_ff, D]        x += W_down( silu(W_gate b) * (W_up b) ),          */
  const void* w_up;     /* [Ld][d_ff, D]        b = N(x) * g_mlp, after the attention residual     */
  const void* w_down;   /* [Ld][D, d_ff]                                                           */
  const void* g_mlp;    /* [Ld][D]              gain of the pre-MLP norm                           */
  const void* g_qnorm;  /* [Ld][hd]             gain of the per-head query norm                    */
  const void* g_knorm;  /* [Ld][hd]             gain of the per-head key norm                      */
  const void* fc_rej;   /* [D, D_in]            COD_F_REJ_PROJECTOR only: fusion map of rejected rows      */
} cod_weights;

/* Mutable drafter state of a batch (device, caller-owned). */
typedef struct {
  void* kv_pool;          /* [Ld][n_pages][n_kv][2][page][hd]  C_l; index 3: 0 = K (rotated), 1 = V */
  int32_t* block_table;   /* [S][max_pages_per_seq]            physical page of each logical page  */
  int32_t* committed_len; /* [S]   L_s; cod_scatter_kv adds the accepted rows                      */
  void* carry_kv;         /* [Ld][max_batch][n_kv][2][k*W][hd] U_l (rows >= carry_len are stale)   */
  int32_t* carry_len;     /* [S]   c_s in 0..k*W, overwritten every round                          */
  int32_t* carry_hist;    /* [S][k] carry_rounds = k > 1 only (else may be NULL): lengths of the k
                                    newest rounds' segments of U_l, oldest first; starts as zeros   */
} cod_state;

/* Output of cod_verify_accept (device, caller-owned). Row ids are s*W + p. */
typedef struct {
  int32_t* accept_len;  /* [S]     m_s                                                      */
  int32_t* bonus;       /* [S]     target[s, m_s]                                           */
  int32_t* row_pos;     /* [S*W]   absolute position L_s + p                                */
  int32_t* commit_slot; /* [S*W]   page*page_size + offset for accepted rows, else -1       */
  int32_t* carry_slot;  /* [S*W]   s*W + (p - m_s) for rejected rows, else -1               */
  int32_t* acc_rows;    /* [S*W]   accepted row ids, increasing; tail filled with -1        */
  int32_t* acc_off;     /* [S+1]   exclusive prefix sums of m_s                             */
  int32_t* rej_rows;    /* [S*W]   rejected row ids, increasing; tail filled with -1        */
  int32_t* rej_off;     /* [S+1]   exclusive prefix sums of W - m_s                         */
} cod_split;

/* Optional float32 taps of cod_draft_round for parity tests (device; any member may be NULL). */
typedef struct {
  float* z;         /* [S*W, D]            normalised fused features of the window rows (rows not
                                           projected in baseline mode are left untouched)   */
  float* attn_out;  /* [Ld][S*W, n_q*hd]   attention output of every layer                  */
  float* x_final;   /* [S*W, D]            residual stream before the final norm            */
  float* top_logit; /* [S*W]               the winning logit of every block row             */
  float* carry_mass;/* [Ld][S, W, n_q]     share of each query's softmax mass that falls on the
                                           carried rows U_l (the diagnostic of Appendix C)  */
} cod_taps;

/* Creates a context on the CURRENT CUDA device and allocates its workspace.
   cfg: host pointer. out: host pointer receiving the handle. */
int cod_create(const cod_config* cfg, cod_ctx** out);
int cod_destroy(cod_ctx* ctx);

/* Records the weight pointers (they must stay valid while the context is used) and
   precomputes F(E_carry) = fc . e_carry: F is linear and bias-free, so
   F(h + E_carry) = F(h) + F(E_carry) (Eq. 2 with Algorithm 1's "add before F").
   bf16 contexts with max_batch * block <= 128 also SNAPSHOT every weight matrix, the embedding
   table included, into tile-major copies inside the workspace (contiguous 16 KB tiles stream
   from HBM measurably faster than 128 separate rows; the workspace grows by the size of the
   copied matrices): after changing weight values in place, call cod_set_weights again. */
int cod_set_weights(cod_ctx* ctx, const cod_weights* w, cod_stream_t stream);

/* Part 1 — greedy verification (Section 2 "Preliminaries"; Algorithm 2 "GreedyVerify").
   draft  [S, W]   device int32: the window's tokens (row 0 = anchor when n_forced = 1).
   target [S, W+1] device int32: the target's greedy token for each window row, so
                   target[s, m_s] is the bonus token.
   m_s = longest prefix with draft == target, the first n_forced (0 or 1) rows always
   accepted. Reads st->committed_len and st->block_table; modifies no state. */
int cod_verify_accept(cod_ctx* ctx, const int32_t* draft, const int32_t* target, int S,
                      int n_forced, const cod_state* st, cod_split* out, cod_stream_t stream);

/* Part 1 at temperature 1 — speculative-sampling verification (Appendix A, "Why verification
   remains valid": the usual target acceptance and residual correction, applied with the drafter's
   actual proposal distribution q). Row p is accepted while u[s,p] * q_tok[s,p] < p_tok[s,p]
   (float32: one rounded product, then the comparison), i.e. with probability min(1, P(x)/Q(x)) for
   the drafted token x; the first n_forced rows are always accepted; the first rejected row ends
   acceptance. p_tok, q_tok, u [S, W] device float32: target and drafter probability of the drafted
   token, and a uniform number in [0, 1). target [S, W+1] device int32: target[s, m] is the token the
   target's sampler supplies after the accepted prefix (drawn from the residual norm(max(0, P - Q)) at
   the first rejected row, from P after a fully accepted window); the library only reads target[s, m_s].
   Output and state use are those of cod_verify_accept. */
int cod_verify_accept_stochastic(cod_ctx* ctx, const int32_t* target, const float* p_tok,
                                 const float* q_tok, const float* u, int S, int n_forced,
                                 const cod_state* st, cod_split* out, cod_stream_t stream);

/* Part 2 — J_l = (K_l(Z), V_l(Z)), Z = F(H + [rejected] E_carry) (Eq. 1-2; Algorithm 1).
   H [S*W, D_in] device. J [Ld][S*W][2][n_kv][hd] device; keys rotated (RoPE) at row_pos.
   COD_CARRY writes every row; COD_BASELINE writes accepted rows only and leaves the
   other rows of J untouched. */
int cod_project_kv(cod_ctx* ctx, const void* H, const cod_split* split, int S, int mode,
                   void* J, cod_stream_t stream);

/* Part 3 — C_l <- [C_l; J_l accepted], U_l <- J_l rejected (Algorithm 1, last steps).
   Copies accepted rows to their page slots and, in COD_CARRY, rejected rows to the carry
   slot; then committed_len[s] += m_s and carry_len[s] = W - m_s (0 in COD_BASELINE). */
int cod_scatter_kv(cod_ctx* ctx, const void* J, const cod_split* split, int S, int mode,
                   cod_state* st, cod_stream_t stream);

/* Part 4 — block attention of one drafter layer over [C_l; U_l; block]
   (Section 2 "Preliminaries"; Algorithm 1 "the next draft reads ctx_l").
   q [S, W, n_q, hd], k_blk / v_blk [S, W, n_kv, hd] device, q and k_blk NOT rotated: the
   call rotates them at positions committed_len[s] + i. No mask; scale 1/sqrt(hd); query
   head g reads KV head g / (n_q / n_kv). use_carry = 0 ignores U_l. With COD_F_QK_NORM
   the caller passes q and k_blk already normalised (cod_draft_round does that itself).
   out [S, W, n_q, hd]. carry_mass (nullable) float [S, W, n_q]: share of softmax mass on
   the carried rows (the diagnostic of Appendix C). */
int cod_block_attn(cod_ctx* ctx, int layer, const void* q, const void* k_blk, const void* v_blk,
                   const cod_state* st, int S, int use_carry, void* out, float* carry_mass,
                   cod_stream_t stream);

/* Part 5 — tied LM head with fused argmax: tok[r] = lowest-index argmax_v Emb[v] . N_f(x[r]).
   x [n_rows, D] device float32 (the residual stream); tok [n_rows] device int32;
   top_logit (nullable) [n_rows] device float. Logits are never materialised. */
int cod_lm_head_argmax(cod_ctx* ctx, const float* x, int n_rows, int32_t* tok, float* top_logit,
                       cod_stream_t stream);

/* Part 5 at temperature 1 — a token per row DRAWN from softmax(Emb . N_f(x[r])) by the Gumbel-max
   rule, tok[r] = lowest-index argmax_v (logit_v - log(-log U(seed, step, r, v))), fused into the
   LM-head contraction like the argmax; logits are never materialised. U is a counter-based uniform
   number: with mix(x) the 32-bit finaliser (x ^= x >> 16; x *= 0x85EBCA6B; x ^= x >> 13;
   x *= 0xC2B2AE35; x ^= x >> 16), h = mix(mix(mix(mix(mix(seed_lo ^ 0x9E3779B9) + seed_hi) + step) + r) + v)
   and U = ((h >> 9) + 0.5) * 2^-23 (the paper fixes no generator; any caller can reproduce this one).
   q_tok (nullable) [n_rows] device float: the soft-max probability of the drawn token — the
   proposal probability Q(x) that cod_verify_accept_stochastic wants next round;
   lse (nullable) [n_rows] device float: log-sum-exp of the row's logits.
   bf16 contexts on the tensor-core kernels only; otherwise COD_ERR_UNSUPPORTED. */
int cod_lm_head_sample(cod_ctx* ctx, const float* x, int n_rows, unsigned long long seed, uint32_t step,
                       int32_t* tok, float* q_tok, float* lse, cod_stream_t stream);

/* Rank of a reference token among the drafter's candidates (Section 5.1 "Target-token recall at
   matched anchors": with ref_tok the target's top token, Recall@k is the share of rows with
   rank < k). rank[r] = number of vocabulary entries v != ref_tok[r] with
   Emb[v] . N_f(x[r]) above Emb[ref_tok[r]] . N_f(x[r]), ties going to the lower index. The count
   is taken inside the LM-head contraction; logits are never materialised. The reference logit is a
   separate float dot product of the same operands, so entries within rounding distance of it may
   fall on either side.
   x [n_rows, D] device float32; ref_tok [n_rows] device int32 (out of range: COD_DEV_BAD_TOKEN,
   token 0 is used); rank [n_rows] device int32; ref_logit (nullable) [n_rows] device float.
   bf16 contexts on the tensor-core kernels only; otherwise COD_ERR_UNSUPPORTED. */
int cod_lm_head_rank(cod_ctx* ctx, const float* x, int n_rows, const int32_t* ref_tok, int32_t* rank,
                     float* ref_logit, cod_stream_t stream);

/* The same argmax as cod_lm_head_argmax for callers that may not allocate device memory: it needs
   no cod_ctx and calls no cudaMalloc / cudaFree or any allocating routine. (The paper has no
   counterpart for this entry point; it exists for integration.) Such callers are, for example, a
   server whose device memory is entirely owned by its own pool, or a latency-critical loop that
   cannot afford cudaMalloc's device-wide synchronisation.
   Its scratch (normalised activations, packed argmax keys) is a fixed array inside the library:
   each GPU that loads the library holds about 2 MiB of it until the process exits.
     emb [vocab, d_model], g_final [d_model]: device, element type `dtype` (cod_dtype);
     x [n_rows, d_model] device float32; tok [n_rows] device int32; top_logit [n_rows] device
     float32 or NULL.
   Limits: n_rows <= 64 and d_model <= 8192, otherwise COD_ERR_TOO_LARGE and nothing is launched.
   All calls on a device share the scratch, which keeps the last call's contents (what must start
   at zero is cleared by the call itself): calls that overlap on the GPU race with each other.
   The first call on a device looks up the scratch's device address with that device current; it
   should be made before any stream capture begins. There is no status word to poll here: a row
   whose contraction did not complete comes back as tok = -1, every other row as an id in [0, vocab). */
int cod_lm_head_argmax_static(const void* emb, const void* g_final, const float* x, int n_rows,
                              int d_model, int vocab, int dtype, float rms_eps, int32_t* tok,
                              float* top_logit, cod_stream_t stream);

/* The whole round: parts 1-3 on (draft, target, H), then one parallel block prediction from
   [bonus, MASK, ...] through every drafter layer, then part 5.
   next_draft [S, W] device int32 = [bonus_s, tok_1, ..., tok_{W-1}].
   Leaves st exactly as cod_verify_accept + cod_project_kv + cod_scatter_kv would.
   taps: host pointer to a struct of device pointers, or NULL. */
int cod_draft_round(cod_ctx* ctx, const int32_t* draft, const int32_t* target, const void* H,
                    int S, int n_forced, int mode, cod_state* st, cod_split* split_out,
                    int32_t* next_draft, const cod_taps* taps, cod_stream_t stream);

/* Copies the sticky device status word to *dev_flags (host) after synchronising the stream;
   clear != 0 also resets it. */
int cod_poll_status(cod_ctx* ctx, uint32_t* dev_flags, int clear, cod_stream_t stream);

/* cod_draft_round at temperature 1: cod_verify_accept_stochastic is its first part, and if q_next is
   non-null the next block is DRAWN by the rule of cod_lm_head_sample (row counter r = s*W + i, the
   given seed and step) instead of taken greedily: next_draft[s, 0] = bonus, next_draft[s, i] = the
   drawn token, q_next [S, W] device float = its soft-max probability (q_next[s, 0] belongs to the
   row-0 draw, which the bonus token replaces). With q_next == NULL the block is the greedy argmax and
   the proposal is a point mass (the next verification then takes q_tok = 1). */
int cod_draft_round_stochastic(cod_ctx* ctx, const int32_t* target, const float* p_tok,
                               const float* q_tok, const float* u, const void* H, int S, int n_forced,
                               int mode, cod_state* st, cod_split* split_out, int32_t* next_draft,
                               const cod_taps* taps, float* q_next, unsigned long long seed,
                               uint32_t step, cod_stream_t stream);

/* Analysis aid — the re-convergence count R of Section 5.2 (the equation defining R), one per
   sequence: R[s] = #{ q in [0, len[s]) : z[s, q+d] == y[s, q] for some d in {-1, 0, +1} with
   0 <= q+d < len[s] }.  z [S, W] device int32: the verifier's top-1 next-token prediction from the
   q-th rejected state; y [S, W] device int32: the token eventually committed at the position that
   prediction refers to; len [S] device int32: rejected suffix length (clamped to [0, W]);
   R [S] device int32. W = cfg.block. It selects nothing and feeds nothing back (as in the paper). */
int cod_reconvergence_count(cod_ctx* ctx, const int32_t* z, const int32_t* y, const int32_t* len, int S,
                            int32_t* R, cod_stream_t stream);

/* Kernel classes for the optional per-kernel timing below. */
enum cod_kernel_class {
  COD_K_VERIFY = 0, /* verify-accept + position tables      */
  COD_K_FC = 1,     /* contraction with F                   */
  COD_K_KV = 2,     /* contraction with K_l, V_l (all l)    */
  COD_K_QKV = 3,    /* Q/K/V of the block rows (per layer)  */
  COD_K_ATTN = 4,   /* block attention (split + combine)    */
  COD_K_OPROJ = 5,  /* output projection (per layer)        */
  COD_K_LMHEAD = 6, /* LM head + argmax                     */
  COD_K_ROWOPS = 7, /* norms, rotations, scatter, read-out  */
  COD_K_MLP = 8,    /* gate/up and down contractions (d_ff > 0) */
  COD_K_CLASSES = 9
};

/* Failure detection (the paper has no counterpart). Every device-side wait of the tensor-core kernels
   (an mbarrier poll in a copy / MMA pipeline) is bounded by the SM cycle counter; when the bound runs out
   the CTA raises COD_DEV_TIMEOUT in the status word, lets what is in flight land, frees its tensor memory
   and returns, so the context stays usable. cod_set_wait_limit sets that bound in SM cycles for the
   context's later launches of the weight-streaming contraction (sm_cycles <= 0: the built-in bound, about
   2 s). */
int cod_set_wait_limit(cod_ctx* ctx, long long sm_cycles);
/* Self-test of that path: while on != 0, the weight-streaming contraction kernel (rounds and calls of up to
   128 rows) requests NO operand copies, so its consumers' waits run out after the wait limit and the calls
   end with COD_DEV_TIMEOUT set and no result (tokens come back as -1). Nothing faults and nothing is left in
   flight. Set a short wait limit first; switch it off again (and clear the status word) before real work. */
int cod_selftest_expire_wait(cod_ctx* ctx, int on);

/* Measurement aid (the paper has no counterpart): while class_mask has bit (1 << k) set,
   every launch of class k is bracketed by CUDA events on the launching stream (at most
   4096 launches are recorded between two calls). class_mask = 0 switches it off.
   Calling it also discards earlier records. */
int cod_profile_enable(cod_ctx* ctx, uint32_t class_mask);
/* Synchronises the recorded events and returns the summed duration and launch count of one
   class since cod_profile_enable. total_ms, launches: host pointers. */
int cod_profile_read(cod_ctx* ctx, int kernel_class, float* total_ms, int32_t* launches);

/* Number of kernels this context has launched since creation (host-side counter). */
int64_t cod_launch_count(const cod_ctx* ctx);

/* Bytes of device workspace the context holds. */
int64_t cod_workspace_bytes(const cod_ctx* ctx);

const char* cod_error_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* COD_H_ */
