// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cod.h"

#define COD_MAX_SPLITS 8          // split-K partial slabs the GEMM workspace can hold
#define COD_MAX_W 128             // largest supported block size
#define COD_L2_KEEP_BYTES (48ll << 20)   // weight bytes of the fc projection asked to stay in L2 between small rounds

// ---------------------------------------------------------------------------- dependent launches
// With few token rows a round is ~45 short kernels, and every kernel is launched with programmatic
// stream serialisation: its CTAs may become resident while the previous kernel of the stream is
// still running, so launch latency and CTA set-up overlap that kernel's tail. cod_pdl_prologue()
// waits until the previous grid has completed and its memory is visible, then (small grids only)
// lets the next grid start launching. Before that call a kernel touches only what no kernel writes:
// its parameters, its own shared and tensor memory and - in the tensor-core GEMMs - the weights,
// whose first tiles are requested ahead of the wait. A GEMM always follows a row-wise kernel, never
// another tensor-memory user, so the tensor memory it allocates ahead of its wait is never needed
// by the grid it waits for.
// For grids of more than ~1000 CTAs the explicit trigger measured slower (the many waiting CTAs of
// the next grid get in the way) and the next grid starts as this one drains; triggering ahead of
// the wait (several grids running ahead) measured slower as well.
__device__ __forceinline__ void cod_pdl_prologue() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (gridDim.x * gridDim.y * gridDim.z <= 1024u) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Drops one 128-byte line (address aligned to 128 bytes) from L2 without writing it back: for scratch data that
// has been read for the last time. Whatever is read there before the next write is indeterminate, and the caller
// orders the drop after every read of the line: the readers synchronise with the dropping thread first, and the
// dropping thread is itself one of the line's readers (the lanes that share a line read it with one instruction).
// Worth its instructions only when the scratch is large enough to be pushed out to HBM under a memory-bound kernel:
// rounds of more token rows than this (one block per row in the kernels that use it).
#define COD_DROP_MIN_ROWS 128
__device__ __forceinline__ void cod_discard_line(const void* p) {
  asm volatile("discard.global.L2 [%0], 128;" ::"l"(p) : "memory");
}

// ---------------------------------------------------------------------------- element access
__device__ __forceinline__ float cod_ld(const float* p) { return *p; }
__device__ __forceinline__ float cod_ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void cod_st(float* p, float v) { *p = v; }
__device__ __forceinline__ void cod_st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// four consecutive elements (pointer aligned to 4 elements)
__device__ __forceinline__ float4 cod_ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 cod_ld4(const __nv_bfloat16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}

__device__ __forceinline__ float cod_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float cod_warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Sum over a thread block (blockDim.x a multiple of 32, at most 1024); result in every thread.
__device__ __forceinline__ float cod_block_sum(float v, float* red /* >= 33 floats of shared */) {
  v = cod_warp_sum(v);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) red[wid] = v;
  __syncthreads();
  if (wid == 0) {
    float t = lane < nw ? red[lane] : 0.f;
    t = cod_warp_sum(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}

// Packed (logit, index) key whose unsigned order is: larger logit first, then lower index.
__device__ __forceinline__ unsigned long long cod_pack_argmax(float v, int idx) {
  unsigned u = __float_as_uint(v);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return (static_cast<unsigned long long>(u) << 32) | static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<unsigned>(idx));
}
__device__ __forceinline__ float cod_unpack_logit(unsigned long long key) {
  unsigned u = static_cast<unsigned>(key >> 32);
  u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
  return __uint_as_float(u);
}
__device__ __forceinline__ int cod_unpack_index(unsigned long long key) {
  return static_cast<int>(0xFFFFFFFFu - static_cast<unsigned>(key & 0xFFFFFFFFull));
}

// ---------------------------------------------------------------------------- GEMM arguments
// C[i, n] = sum_k A[row(i), k] * B[n, k]   (A: activations, B: weights, both K contiguous)
struct GemmSeg {
  const void* B;  // [N, K]
  int N;
  const void* Bt; // optional tile-major copy of B (see cod_launch_retile); null: read B itself
};
struct GemmArgs {
  const void* A;          // [*, K] with row stride lda
  int lda;
  const int* a_rows;      // optional gather list: row(i) = a_rows[i]; else row(i) = i
  const int* n_rows_dev;  // optional device count of valid rows (<= n_rows)
  int rows_gate;          // n_rows_dev only gates the launch: all n_rows rows if it is positive, none if it is zero
  const int* group_split_dev;  // paired kernel, two segments: rows [0, *g) meet segment 0, rows [*g, n_rows) segment 1, both
                          // write the SAME columns [0, seg[0].N) (a contraction grouped by row); null: segments side by side
  int n_rows;             // rows (or their upper bound when n_rows_dev is set)
  int K;
  GemmSeg seg[3];         // weight segments laid side by side along N
  int n_seg;
  float* C;               // [splits][n_rows][ldc] float partial sums
  int ldc;
  int splits;             // split-K factor (1 = none)
  int n_acc;              // paired kernel: accumulators per CTA pair (1 or 2); 0 = let the launcher choose
  unsigned long long* amax;  // if non-null: per-row packed argmax over N instead of storing C
  // sampling form of the argmax epilogue (tensor-core kernels only): keys carry logit + Gumbel noise and
  // every 128-row weight tile also leaves (m, sum exp(logit - m)) per token row in lse_part[tile][n_rows]
  float2* lse_part;       // null: plain argmax
  uint32_t sample_state;  // hash state after seed and step
  int klass;              // cod_kernel_class, for the optional timing
  // rank form (k_gemm_tc only): rank_out[i] += number of weight rows n != rank_tok[i] whose product with
  // row i lies above rank_ref[i] (ties: lower n first); nothing else is stored
  const float* rank_ref;
  const int32_t* rank_tok;
  unsigned int* rank_out;
};

#define COD_PROF_SLOTS 4096

struct cod_ctx {
  cod_config cfg;
  cod_weights w;
  bool has_weights;
  int device;
  int D, D_in, kvw, qw, R_max, half;
  int split_len, max_splits;   // attention split-KV (plain-FMA kernel)
  int tc_split_len, tc_max_parts;  // attention split-KV (tensor-core kernel); 0 parts = not usable
  void* zero_page;             // 16 x 128 bf16 zeros (stands in for pages past the end of a split)
  int n_sm;
  bool force_simt;             // COD_F_NO_TENSOR_CORES: plain-FMA kernels only
  bool pdl;                    // launch kernels as programmatic dependents of their predecessor in the stream
  int64_t launches;
  size_t ws_bytes;
  char* ws;
  // carved out of ws
  uint32_t* status;
  float* inv_freq;             // [hd/2]  theta^(-2j/hd), rounded from double
  double* inv_freq_d;          // [hd/2]
  float* fcE;                  // [D]     F(E_carry)
  float* rope_win;             // [R_max][hd]  cos | sin of the window rows' positions
  float* rope_blk;             // [R_max][hd]  cos | sin of the block rows' positions
  void* hmid;                  // [R, d_ff] activated MLP rows (storage type), d_ff > 0 only
  float2* lse_part;            // [ceil(vocab / 128)][R] soft-max partials of the sampling LM head
  void* emb_tiled;             // tile-major copy of the embedding table (bf16 tensor-core path), made by cod_set_weights
  // tile-major copies of the other weight matrices, for rounds of up to 128 rows (null where the matrix
  // does not cut into whole 128-row tiles per layer, or for large-batch-only contexts); per layer l a
  // matrix [N, K] starts at l * cod_retile_bytes(N, K)
  struct { char *fc, *fc_rej, *wk, *wv, *wq, *wo, *w_gate, *w_up, *w_down; } wt;
  float* gemm_out;             // split-K / unfused GEMM results
  int carry_cap;               // rows of one (layer, sequence, head, K|V) carry slot: carry_rounds * block
  int* carry_base;             // [max_batch] rows of U kept from earlier rounds (carry_rounds > 1), else null
  int* carry_drop;             // [max_batch] rows of U that leave this round (carry_rounds > 1), else null
  float* gemm_out2;            // a second, small slab buffer for the side branch of the round (null: no side branch)
  int* attn_order;             // [max_batch * tc_max_parts] longest-first work list of the tensor-core attention
  int* attn_counter;           // work units the persistent attention CTAs have taken beyond their first (zero between launches)
  bool attn_order_stale;       // the lengths may have changed since the list was built
  int side_rows;               // the side branch is used for rounds of at most this many rows
  cudaStream_t side;           // side branch of the round: the first layer's embedding / Q/K/V chain
  cudaEvent_t ev_fork, ev_join;
  size_t gemm_out_floats;
  void* hc;                    // [R_max, D_in] accepted rows of H packed densely (baseline mode)
  long long wait_limit;        // SM cycles a bounded device wait may last (0: the built-in limit, about 2 s)
  int attn_one_item_ctas;      // 1: work-list attention as one CTA per item (the persistent form off; for A/B runs)
  int attn_persistent;         // 1: the persistent form whatever the geometry
  bool attn_run_ahead;         // false while the next attention launch follows a kernel that writes the KV state or the lengths
  int selftest_skip_copies;    // cod_selftest_expire_wait: single-CTA contractions request no operands
  int* perm;                  // [R] window rows in the order accepted-first (grouped contraction of the separate projector)
  void* z;                     // [R_max, D]
  float* x;                    // [R_max, D]   residual stream
  void* a;                     // [R_max, D]   normalised activations
  void* q;                     // [R_max, qw]
  void* kb;                    // [R_max, kvw]
  void* vb;                    // [R_max, kvw]
  void* o;                     // [R_max, qw]
  float* attn_o;               // [S][n_kv][splits][M][hd]
  float* attn_ml;              // [S][n_kv][splits][M][4]  (m, l, l_carry, -)
  unsigned long long* amax;    // [R_max]
  int32_t* tok;                // [R_max]
  cod_split sp;                // internal split arrays (used when the caller passes none)
  // optional per-kernel timing
  uint32_t prof_mask;
  int prof_n;
  cudaEvent_t* prof_ev;        // [2 * COD_PROF_SLOTS], created at cod_create
  unsigned char* prof_class;   // [COD_PROF_SLOTS]
};

// Brackets the launches made inside its scope with two events when the class is being timed.
struct ProfScope {
  cod_ctx* c; cudaStream_t st; int slot;
  ProfScope(cod_ctx* c_, int klass, cudaStream_t st_) : c(c_), st(st_), slot(-1) {
    if ((c->prof_mask >> klass) & 1u) {
      if (c->prof_n < COD_PROF_SLOTS) {
        slot = c->prof_n++;
        c->prof_class[slot] = static_cast<unsigned char>(klass);
        cudaEventRecord(c->prof_ev[2 * slot], st);
      }
    }
  }
  ~ProfScope() { if (slot >= 0) cudaEventRecord(c->prof_ev[2 * slot + 1], st); }
};

template <typename... KArgs, typename... Args>
inline cudaError_t cod_launch_pdl(const cod_ctx* c, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = c->pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------- launchers
// Every launcher enqueues on `st`, bumps ctx->launches, and returns a cod_status.
// p_tok / q_tok / u all null: greedy rule (draft == target); all non-null: speculative sampling (draft unused)
int cod_launch_verify(cod_ctx* c, const int32_t* draft, const int32_t* target, int S, int n_forced,
                      const cod_state* state, const cod_split* out, cudaStream_t st, const float* p_tok = nullptr,
                      const float* q_tok = nullptr, const float* u = nullptr);
int cod_launch_gemm(cod_ctx* c, const GemmArgs& g, cudaStream_t st);
int cod_launch_gemm_simt(cod_ctx* c, const GemmArgs& g, cudaStream_t st);
bool cod_gemm_tc_supported(const cod_ctx* c, const GemmArgs& g);
bool cod_gemm_tc2_supported(const cod_ctx* c, const GemmArgs& g);
// Tile plan of the paired kernel for n_out weight rows, K and `rows` token rows: split-K factor and
// accumulators per pair with the least modelled time (no split is left empty). fixed_splits > 0 pins
// the split-K factor and only chooses the accumulators.
void cod_plan_gemm_tc2(int n_sm, int n_out, int K, int rows, int max_splits, int fixed_splits, int* splits,
                       int* n_acc);
int cod_launch_gemm_tc2(cod_ctx* c, const GemmArgs& g, cudaStream_t st);
bool cod_attn_tc_supported(const cod_ctx* c);
int cod_launch_attn_tc(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb, const cod_state* stt,
                       int S, int use_carry, void* out, float* tap, float* mass, cudaStream_t st);
int cod_launch_gemm_tc(cod_ctx* c, const GemmArgs& g, cudaStream_t st);
int cod_launch_attn_simt(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb,
                         const cod_state* stt, int S, int use_carry, void* out, float* tap, float* mass,
                         cudaStream_t st);
// cos/sin tables of the block rows only, at positions committed_len[s] + i
int cod_launch_reconvergence(cod_ctx* c, const int32_t* z, const int32_t* y, const int32_t* len, int S,
                             int32_t* R, cudaStream_t st);
int cod_launch_finalize_sample(cod_ctx* c, int R, uint32_t state, int32_t* tok, float* q_tok, float* lse,
                               cudaStream_t st, const int32_t* bonus = nullptr, int32_t* next_draft = nullptr);
uint32_t cod_sample_state(unsigned long long seed, uint32_t step);   // hash state after seed and step
// carry_rounds > 1: drops the oldest round's rows of U, moves the kept ones to the front, shifts the history
int cod_launch_carry_age(cod_ctx* c, const cod_split* sp, int S, int mode, const cod_state* st, cudaStream_t stream);
// Copies a bf16 matrix [N, K] into 16 KB tiles of 128 rows x 64 columns, tile (row tile, k block) at
// ((row tile) * ceil(K / 64) + k block) * 16 KB, each tile already in the 128-byte-swizzled order the
// tensor core reads from shared memory (rows and columns beyond the matrix are zero): a GEMM then
// fetches its weight tiles as contiguous 16 KB bulk copies, which stream ~4 % faster from DRAM than
// 128 separate 128-byte rows.
int cod_launch_retile(cod_ctx* c, const void* B, int N, int K, void* Bt, cudaStream_t st);
size_t cod_retile_bytes(int N, int K);
int cod_launch_rope_blk_only(cod_ctx* c, const int32_t* committed_len, int S, cudaStream_t st);
int cod_launch_fcE(cod_ctx* c, cudaStream_t st);
int cod_launch_gather_rows(cod_ctx* c, const void* src, const int* rows, const int* n_dev, int n_max, int width,
                           void* dst, cudaStream_t st);
// dst = src rows in the order acc_rows[0 .. *n_acc) then rej_rows[0 .. R - *n_acc); perm receives that order
int cod_launch_gather_grouped(cod_ctx* c, const void* src, const cod_split* sp, int S, int R, int width, void* dst, int* perm,
                              cudaStream_t st);
int cod_launch_fc_finish(cod_ctx* c, const float* part, int splits, int n_rows, const int* n_rows_dev,
                         const int* a_rows, const int* carry_slot, float* tap_z, cudaStream_t st, int ldp = 0, int dense_base = 0, int z_by_row = 0);   // ldp: row stride of part (0 = D; 2 D = F h | F_rej h)
// dest_state == nullptr: write J; else write the pool / carry slot directly
int cod_launch_kv_finish(cod_ctx* c, const float* part, int splits, int n_rows, const int* n_rows_dev,
                         const int* a_rows, const cod_split* sp, void* J, const cod_state* dest_state,
                         int R_total, cudaStream_t st, int dense_base = 0);
int cod_launch_scatter(cod_ctx* c, const void* J, const cod_split* sp, int S, int mode,
                       const cod_state* state, cudaStream_t st);
int cod_launch_update_lens(cod_ctx* c, const cod_split* sp, int S, int mode, const cod_state* state,
                           cudaStream_t st);
// sp non-null: the kernel also performs cod_launch_update_lens's update (inside a round)
int cod_launch_embed_norm(cod_ctx* c, const int32_t* bonus, int S, cudaStream_t st, const cod_split* sp = nullptr,
                          int mode = 0, const cod_state* ds = nullptr);
// reference logits ref[r] = a[r] . Emb[tok[r]] of the rank form; also sanitises the tokens and zeroes the counts
int cod_launch_rank_ref(cod_ctx* c, int n_rows, const int32_t* ref_tok, float* ref, int32_t* tok_clean,
                        int32_t* rank, cudaStream_t st);
int cod_launch_qkv_finish(cod_ctx* c, const float* part, int splits, int R, int layer, cudaStream_t st);
int cod_launch_swiglu_finish(cod_ctx* c, const float* part, int splits, int R, cudaStream_t st);
int cod_launch_rope_qk(cod_ctx* c, const void* q, const void* k, const int32_t* committed_len, int S,
                       cudaStream_t st);  // standalone attention entry: rotate into c->q / c->kb
int cod_launch_attn(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb,
                    const cod_state* state, int S, int use_carry, void* out, float* tap_out,
                    float* carry_mass, cudaStream_t st);
// x += sum of partials (if part != nullptr); a = N(x) * gain; optional copy of x to tap_x
int cod_launch_resid_norm(cod_ctx* c, const float* part, int splits, int R, float* x, const void* gain,
                          float* tap_x, cudaStream_t st);
int cod_launch_finalize(cod_ctx* c, int R, int W, const int32_t* bonus, int32_t* tok, int32_t* next_draft,
                        float* top_logit, cudaStream_t st);

#define COD_CHECK_LAUNCH(c)                                   \
  do {                                                        \
    (c)->launches++;                                          \
    if (cudaPeekAtLastError() != cudaSuccess) return COD_ERR_CUDA; \
  } while (0)
