// The C ABI: argument validation, workspace, and the order of kernels in one round.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "cod_internal.cuh"

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t esize(const cod_ctx* c) { return c->cfg.dtype == COD_BF16 ? 2 : 4; }
inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

struct Carver {
  char* base;
  size_t off;
  template <typename P>
  void take(P*& ptr, size_t bytes) {
    off = align_up(off, 256);
    if (base) ptr = reinterpret_cast<P*>(base + off);
    off += bytes;
  }
};

// Lays out the workspace; with c->ws == nullptr it only measures.
size_t carve(cod_ctx* c) {
  const cod_config& f = c->cfg;
  const size_t R = c->R_max, es = esize(c), D = c->D;
  Carver cv{c->ws, 0};
  cv.take(c->status, 256);
  cv.take(c->inv_freq_d, sizeof(double) * c->half);
  cv.take(c->inv_freq, sizeof(float) * c->half);
  cv.take(c->fcE, sizeof(float) * D);
  cv.take(c->rope_win, sizeof(float) * R * f.head_dim);
  cv.take(c->rope_blk, sizeof(float) * R * f.head_dim);
  size_t widest = D;
  widest = widest > static_cast<size_t>(2 * f.n_layers * c->kvw) ? widest : static_cast<size_t>(2 * f.n_layers * c->kvw);
  widest = widest > static_cast<size_t>(c->qw + 2 * c->kvw) ? widest : static_cast<size_t>(c->qw + 2 * c->kvw);
  widest = widest > static_cast<size_t>(2 * f.d_ff) ? widest : static_cast<size_t>(2 * f.d_ff);
  if ((f.flags & COD_F_REJ_PROJECTOR) && widest < 2 * D) widest = 2 * D;
  c->gemm_out_floats = static_cast<size_t>(COD_MAX_SPLITS) * R * widest;
  cv.take(c->gemm_out, sizeof(float) * c->gemm_out_floats);
  // the side branch (first layer's Q/K/V chain next to the context projection) pays off where the
  // round is a chain of short, latency-bound kernels: up to 128 rows
  c->side_rows = static_cast<int>(R < 128 ? R : 128);
  cv.take(c->gemm_out2, sizeof(float) * COD_MAX_SPLITS * c->side_rows * (c->qw + 2 * c->kvw));
  cv.take(c->hc, es * R * c->D_in);
  cv.take(c->perm, sizeof(int) * R);
  cv.take(c->z, es * R * D);
  cv.take(c->x, sizeof(float) * R * D);
  cv.take(c->a, es * R * D);
  cv.take(c->q, es * R * c->qw);
  cv.take(c->kb, es * R * c->kvw);
  cv.take(c->vb, es * R * c->kvw);
  cv.take(c->o, es * R * c->qw);
  if (f.d_ff > 0) cv.take(c->hmid, es * R * f.d_ff);
  const size_t M = static_cast<size_t>(f.block) * (f.n_q_heads / f.n_kv_heads);
  const size_t per_head = static_cast<size_t>(c->max_splits > c->tc_max_parts ? c->max_splits : c->tc_max_parts);
  const size_t parts = static_cast<size_t>(f.max_batch) * f.n_kv_heads * per_head * M;
  cv.take(c->zero_page, 4096);
  cv.take(c->attn_o, sizeof(float) * parts * f.head_dim);
  cv.take(c->attn_ml, sizeof(float) * parts * 4);
  if (c->tc_max_parts > 0) cv.take(c->attn_order, sizeof(int) * f.max_batch * c->tc_max_parts);
  cv.take(c->attn_counter, 256);
  if (c->carry_cap > f.block) {
    cv.take(c->carry_base, sizeof(int) * f.max_batch);
    cv.take(c->carry_drop, sizeof(int) * f.max_batch);
  }
  cv.take(c->amax, sizeof(unsigned long long) * R);
  cv.take(c->lse_part, sizeof(float2) * R * ((static_cast<size_t>(f.vocab) + 127) / 128));
  // rounds of up to 128 rows stream every weight matrix through the single-CTA kernel: tile-major copies
  // (conditions on the configuration only: the measuring pass of this function assigns no pointers)
  const bool tile_ok = f.dtype == COD_BF16 && !(f.flags & COD_F_NO_TENSOR_CORES) && f.d_model % 8 == 0 &&
                       (f.d_target * f.n_cap) % 8 == 0;
  // (contexts sized for more than 128 rows run the paired kernel, which reads the caller's matrices: no copies)
  const bool tile_all = tile_ok && f.max_batch * f.block <= 128;
  if (tile_all) cv.take(c->emb_tiled, cod_retile_bytes(f.vocab, f.d_model));
  if (tile_all) {
    const int Ld = f.n_layers, kvw = c->kvw, qw = c->qw, Dm = c->D;
    if (Dm % 128 == 0) cv.take(c->wt.fc, cod_retile_bytes(Dm, c->D_in));
    if (Dm % 128 == 0 && (f.flags & COD_F_REJ_PROJECTOR)) cv.take(c->wt.fc_rej, cod_retile_bytes(Dm, c->D_in));
    if (kvw % 128 == 0) { cv.take(c->wt.wk, Ld * cod_retile_bytes(kvw, Dm)); cv.take(c->wt.wv, Ld * cod_retile_bytes(kvw, Dm)); }
    if (qw % 128 == 0) cv.take(c->wt.wq, Ld * cod_retile_bytes(qw, Dm));
    if (Dm % 128 == 0 && qw % 8 == 0) cv.take(c->wt.wo, Ld * cod_retile_bytes(Dm, qw));
    if (f.d_ff > 0 && f.d_ff % 128 == 0) {
      cv.take(c->wt.w_gate, Ld * cod_retile_bytes(f.d_ff, Dm));
      cv.take(c->wt.w_up, Ld * cod_retile_bytes(f.d_ff, Dm));
      if (Dm % 128 == 0) cv.take(c->wt.w_down, Ld * cod_retile_bytes(Dm, f.d_ff));
    }
  }
  cv.take(c->tok, sizeof(int32_t) * R);
  cv.take(c->sp.accept_len, sizeof(int32_t) * f.max_batch);
  cv.take(c->sp.bonus, sizeof(int32_t) * f.max_batch);
  cv.take(c->sp.row_pos, sizeof(int32_t) * R);
  cv.take(c->sp.commit_slot, sizeof(int32_t) * R);
  cv.take(c->sp.carry_slot, sizeof(int32_t) * R);
  cv.take(c->sp.acc_rows, sizeof(int32_t) * R);
  cv.take(c->sp.acc_off, sizeof(int32_t) * (f.max_batch + 1));
  cv.take(c->sp.rej_rows, sizeof(int32_t) * R);
  cv.take(c->sp.rej_off, sizeof(int32_t) * (f.max_batch + 1));
  return align_up(cv.off, 256);
}

bool split_has_null(const cod_split* s) {
  return !s || !s->accept_len || !s->bonus || !s->row_pos || !s->commit_slot || !s->carry_slot || !s->acc_rows ||
         !s->acc_off || !s->rej_rows || !s->rej_off;
}
bool state_has_null(const cod_state* s) {
  return !s || !s->kv_pool || !s->block_table || !s->committed_len || !s->carry_kv || !s->carry_len;
}

// split-K factor so that (feature tiles x splits) fills the machine; partial slabs must fit
int pick_splits(const cod_ctx* c, int n_out, int K, int rows) {
  if (c->cfg.dtype != COD_BF16 || c->force_simt) return 1;
  if (rows > 128) {                         // the paired kernel: its own time model picks tiles and splits
    int splits, n_acc;
    cod_plan_gemm_tc2(c->n_sm, n_out, K, rows, COD_MAX_SPLITS, 0, &splits, &n_acc);
    return splits;
  }
  const int tiles = (n_out + 127) / 128;
  const int kb = (K + 63) / 64;
  // up to 32 token rows two CTAs fit on an SM (the launcher keeps their rings small): aim for two waves' worth
  int splits = (rows <= 32 ? 2 * c->n_sm : c->n_sm) / tiles;
  if (splits > COD_MAX_SPLITS) splits = COD_MAX_SPLITS;
  if (splits > kb / 4) splits = kb / 4;
  if (splits < 1) splits = 1;
  const int per = (kb + splits - 1) / splits;
  return (kb + per - 1) / per;            // no empty split
}

bool hist_missing(const cod_ctx* c, const cod_state* s) { return c->carry_cap > c->cfg.block && !s->carry_hist; }

int check_S(const cod_ctx* c, int S) { return (S >= 1 && S <= c->cfg.max_batch) ? COD_OK : COD_ERR_INVALID_ARG; }

}  // namespace

int cod_launch_gemm(cod_ctx* c, const GemmArgs& g, cudaStream_t st) {
  ProfScope prof(c, g.klass, st);
  if (!c->force_simt && cod_gemm_tc2_supported(c, g)) return cod_launch_gemm_tc2(c, g, st);
  if (!c->force_simt && cod_gemm_tc_supported(c, g)) return cod_launch_gemm_tc(c, g, st);
  return cod_launch_gemm_simt(c, g, st);
}

int cod_launch_attn(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb, const cod_state* state,
                    int S, int use_carry, void* out, float* tap_out, float* carry_mass, cudaStream_t st) {
  ProfScope prof(c, COD_K_ATTN, st);
  if (cod_attn_tc_supported(c)) return cod_launch_attn_tc(c, layer, q, kb, vb, state, S, use_carry, out, tap_out, carry_mass, st);
  return cod_launch_attn_simt(c, layer, q, kb, vb, state, S, use_carry, out, tap_out, carry_mass, st);
}

extern "C" {

int cod_create(const cod_config* cfg, cod_ctx** out) {
  if (!cfg || !out) return COD_ERR_INVALID_ARG;
  *out = nullptr;
  const cod_config& f = *cfg;
  if (f.d_target < 1 || f.n_cap < 1 || f.d_model < 1 || f.n_layers < 1 || f.n_q_heads < 1 || f.n_kv_heads < 1 ||
      f.head_dim < 1 || f.vocab < 2 || f.block < 1 || f.page_size < 1 || f.max_batch < 1 ||
      f.max_pages_per_seq < 1 || f.n_pages < 1)
    return COD_ERR_INVALID_ARG;
  if (f.dtype != COD_F32 && f.dtype != COD_BF16) return COD_ERR_INVALID_ARG;
  if (f.mask_token_id < 0 || f.mask_token_id >= f.vocab) return COD_ERR_INVALID_ARG;
  if (f.n_q_heads % f.n_kv_heads) return COD_ERR_INVALID_ARG;
  if (f.d_model != f.n_q_heads * f.head_dim) return COD_ERR_INVALID_ARG;
  if (f.attn_split_len < 0 || f.attn_split_len % 32) return COD_ERR_INVALID_ARG;
  if (!(f.rope_theta > 0.f) || !(f.rms_eps >= 0.f)) return COD_ERR_INVALID_ARG;
  if (f.head_dim != 64 && f.head_dim != 128) return COD_ERR_UNSUPPORTED;
  if (f.block > COD_MAX_W || f.block * (f.n_q_heads / f.n_kv_heads) > 128) return COD_ERR_UNSUPPORTED;
  if ((f.d_target * f.n_cap) % 8 || f.d_model % 8 || f.d_model > 32768) return COD_ERR_UNSUPPORTED;
  if ((f.n_kv_heads * f.head_dim) % 64) return COD_ERR_UNSUPPORTED;
  if (f.d_ff < 0 || f.carry_rounds < 0 || f.carry_rounds > 8) return COD_ERR_INVALID_ARG;
  if (f.d_ff % 64) return COD_ERR_UNSUPPORTED;
  if ((f.flags & COD_F_NO_CARRY_EMBED) && (f.flags & COD_F_REJ_PROJECTOR)) return COD_ERR_INVALID_ARG;
  if ((f.flags & COD_F_REJ_PROJECTOR) && f.d_model % 64) return COD_ERR_UNSUPPORTED;   // F | F_rej share one contraction   // gate and up share one contraction: tiles must not straddle them
  if (static_cast<int64_t>(f.n_pages) * f.page_size > (1ll << 31) - 1) return COD_ERR_UNSUPPORTED;

  cod_ctx* c = new (std::nothrow) cod_ctx();
  if (!c) return COD_ERR_ALLOC;
  memset(c, 0, sizeof(*c));
  c->cfg = f;
  if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return COD_ERR_CUDA; }
  c->D = f.d_model;
  c->D_in = f.d_target * f.n_cap;
  c->kvw = f.n_kv_heads * f.head_dim;
  c->qw = f.n_q_heads * f.head_dim;
  c->R_max = f.max_batch * f.block;
  c->half = f.head_dim / 2;
  c->force_simt = (f.flags & COD_F_NO_TENSOR_CORES) != 0;
  c->attn_one_item_ctas = (f.flags & COD_F_ATTN_ONE_ITEM_CTAS) != 0;
  c->attn_persistent = (f.flags & COD_F_ATTN_PERSISTENT) != 0;
  c->attn_run_ahead = true;
  c->carry_cap = (f.carry_rounds > 1 ? f.carry_rounds : 1) * f.block;
  if (cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess || c->n_sm < 1) c->n_sm = 148;
  c->split_len = f.attn_split_len > 0 ? f.attn_split_len : 512;
  const int64_t max_keys = static_cast<int64_t>(f.max_pages_per_seq) * f.page_size + c->carry_cap + f.block;
  c->max_splits = static_cast<int>((max_keys + c->split_len - 1) / c->split_len);

  {
    // tensor-core attention: keys of the paged region per CTA, and partial slots per (sequence, head)
    const int64_t cap = static_cast<int64_t>(f.max_pages_per_seq) * f.page_size;
    int64_t sl;
    if (f.attn_split_len > 0) sl = (f.attn_split_len + 127) / 128 * 128 > 4096 ? 4096 : (f.attn_split_len + 127) / 128 * 128;
    else {
      // large batches: enough parts to keep every SM fed for several waves
      sl = (cap * f.max_batch * f.n_kv_heads / (8 * static_cast<int64_t>(c->n_sm)) + 127) / 128 * 128;
      if (sl < 256) sl = 256;   // fewer, longer parts beat more CTAs at batch 1 (measured at 2K context)
      if (sl > 2048) sl = 2048;
      // grids that stay several waves deep run their parts longest first (k_attn_order), which evens out
      // the last wave by itself: there, parts twice as long (fewer partial results to merge) measured
      // faster (batch 32, contexts 0.9K..8K: 140 -> 133 us per layer)
      {
        int64_t sl2 = (cap * f.max_batch * f.n_kv_heads / (4 * static_cast<int64_t>(c->n_sm)) + 127) / 128 * 128;
        if (sl2 > 4096) sl2 = 4096;
        if (sl2 > sl && static_cast<int64_t>(f.max_batch) * f.n_kv_heads * ((cap + sl2 - 1) / sl2 + 1) > 4 * static_cast<int64_t>(c->n_sm))
          sl = sl2;
      }
      // small batches: all parts in ONE wave of two CTAs per SM if at least four parts per
      // (sequence, head) fit (a second, mostly empty wave cost 10 % at 4 x 32K keys)
      const int64_t per_seq = 2 * static_cast<int64_t>(c->n_sm) / (static_cast<int64_t>(f.max_batch) * f.n_kv_heads);
      if (per_seq >= 4) {
        int64_t one_wave = ((cap + per_seq - 1) / per_seq + 127) / 128 * 128;
        if (one_wave < 256) one_wave = 256;
        if (one_wave <= 4096) sl = one_wave;
      }
    }
    c->tc_split_len = static_cast<int>(sl);
    c->tc_max_parts = static_cast<int>((cap + sl - 1) / sl + 1);
  }
  c->ws = nullptr;
  c->ws_bytes = carve(c);
  if (cudaMalloc(&c->ws, c->ws_bytes) != cudaSuccess) { cudaGetLastError(); delete c; return COD_ERR_ALLOC; }
  carve(c);
  bool ok = cudaMemset(c->ws, 0, c->ws_bytes) == cudaSuccess;
  double* fr = static_cast<double*>(malloc(sizeof(double) * c->half));
  float* frf = static_cast<float*>(malloc(sizeof(float) * c->half));
  if (!fr || !frf) ok = false;
  if (ok) {
    for (int j = 0; j < c->half; ++j) {
      fr[j] = pow(static_cast<double>(f.rope_theta), -2.0 * j / f.head_dim);
      frf[j] = static_cast<float>(fr[j]);
    }
    ok = cudaMemcpy(c->inv_freq_d, fr, sizeof(double) * c->half, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(c->inv_freq, frf, sizeof(float) * c->half, cudaMemcpyHostToDevice) == cudaSuccess;
  }
  free(fr);
  free(frf);
  c->prof_ev = static_cast<cudaEvent_t*>(calloc(2 * COD_PROF_SLOTS, sizeof(cudaEvent_t)));
  c->prof_class = static_cast<unsigned char*>(calloc(COD_PROF_SLOTS, 1));
  if (!c->prof_ev || !c->prof_class) ok = false;
  if (ok) ok = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess &&
               cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < 2 * COD_PROF_SLOTS; ++i) ok = cudaEventCreate(&c->prof_ev[i]) == cudaSuccess;
  if (!ok) { cudaFree(c->ws); cudaGetLastError(); free(c->prof_ev); free(c->prof_class); delete c; return COD_ERR_CUDA; }
  *out = c;
  return COD_OK;
}

int cod_destroy(cod_ctx* c) {
  if (!c) return COD_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  cudaFree(c->ws);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->side) cudaStreamDestroy(c->side);
  for (int i = 0; i < 2 * COD_PROF_SLOTS; ++i) cudaEventDestroy(c->prof_ev[i]);
  free(c->prof_ev);
  free(c->prof_class);
  delete c;
  return COD_OK;
}

int cod_set_weights(cod_ctx* c, const cod_weights* w, cod_stream_t stream) {
  if (!c || !w) return COD_ERR_INVALID_ARG;
  const void* ps[] = {w->fc, w->e_carry, w->g_hidden, w->wk, w->wv, w->wq, w->wo, w->g_attn, w->g_final, w->emb};
  for (const void* p : ps)
    if (!p || misaligned(p)) return COD_ERR_INVALID_ARG;
  if (c->cfg.d_ff > 0)
    for (const void* p : {w->w_gate, w->w_up, w->w_down, w->g_mlp})
      if (!p || misaligned(p)) return COD_ERR_INVALID_ARG;
  if (c->cfg.flags & COD_F_QK_NORM)
    for (const void* p : {w->g_qnorm, w->g_knorm})
      if (!p || misaligned(p)) return COD_ERR_INVALID_ARG;
  if ((c->cfg.flags & COD_F_REJ_PROJECTOR) && (!w->fc_rej || misaligned(w->fc_rej))) return COD_ERR_INVALID_ARG;
  c->w = *w;
  c->has_weights = true;
  c->pdl = false;
  if (c->emb_tiled) {
    cudaStream_t ss = static_cast<cudaStream_t>(stream);
    int rc = cod_launch_retile(c, w->emb, c->cfg.vocab, c->D, c->emb_tiled, ss);
    const cod_config& f = c->cfg;
    // a stacked matrix [Ld][N, K] whose N is a whole number of tiles re-tiles as one matrix of Ld * N rows
    auto all = [&](const void* src, char* dst, int N, int K, int layers) {
      if (dst && rc == COD_OK) rc = cod_launch_retile(c, src, layers * N, K, dst, ss);
    };
    all(w->fc, c->wt.fc, c->D, c->D_in, 1);
    all(w->fc_rej, c->wt.fc_rej, c->D, c->D_in, 1);
    all(w->wk, c->wt.wk, c->kvw, c->D, f.n_layers);
    all(w->wv, c->wt.wv, c->kvw, c->D, f.n_layers);
    all(w->wq, c->wt.wq, c->qw, c->D, f.n_layers);
    all(w->wo, c->wt.wo, c->D, c->qw, f.n_layers);
    all(w->w_gate, c->wt.w_gate, f.d_ff, c->D, f.n_layers);
    all(w->w_up, c->wt.w_up, f.d_ff, c->D, f.n_layers);
    all(w->w_down, c->wt.w_down, c->D, f.d_ff, f.n_layers);
    if (rc != COD_OK) return rc;
  }
  return cod_launch_fcE(c, static_cast<cudaStream_t>(stream));
}

int cod_verify_accept(cod_ctx* c, const int32_t* draft, const int32_t* target, int S, int n_forced,
                      const cod_state* st, cod_split* out, cod_stream_t stream) {
  if (!c || !draft || !target || !st || !st->committed_len || !st->block_table || split_has_null(out))
    return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK || n_forced < 0 || n_forced > 1) return COD_ERR_INVALID_ARG;
  c->pdl = true;
  return cod_launch_verify(c, draft, target, S, n_forced, st, out, static_cast<cudaStream_t>(stream));
}

int cod_verify_accept_stochastic(cod_ctx* c, const int32_t* target, const float* p_tok, const float* q_tok,
                                 const float* u, int S, int n_forced, const cod_state* st, cod_split* out,
                                 cod_stream_t stream) {
  if (!c || !target || !p_tok || !q_tok || !u || !st || !st->committed_len || !st->block_table || split_has_null(out))
    return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK || n_forced < 0 || n_forced > 1) return COD_ERR_INVALID_ARG;
  c->pdl = true;
  return cod_launch_verify(c, nullptr, target, S, n_forced, st, out, static_cast<cudaStream_t>(stream), p_tok, q_tok, u);
}

// fc and K/V contractions of the kept rows; the finish kernel writes J or the state.
static int project_impl(cod_ctx* c, const void* H, const cod_split* sp, int S, int mode, void* J,
                        const cod_state* dest, float* tap_z, cudaStream_t st) {
  const cod_config& f = c->cfg;
  const int R = S * f.block;
  // The baseline drafter projects accepted rows only. Rounds of up to 128 rows run on the weight-streaming
  // kernel, where extra token columns cost nothing: there the baseline contracts all R rows in place (no
  // packing pass, the same launches as the carry round) and the finish kernels keep the accepted ones; with no
  // accepted row at all both contractions still leave at once. Larger rounds pack the accepted rows first.
  const bool dense_base = mode == COD_BASELINE && R <= 128 && c->cfg.dtype == COD_BF16 && !c->force_simt;
  const int* a_rows = mode == COD_BASELINE && !dense_base ? sp->acc_rows : nullptr;
  const int* n_dev = mode == COD_BASELINE ? sp->acc_off + S : nullptr;
  int rc;

  if (a_rows) {   // baseline: pack the accepted rows, then the same dense kernels on fewer rows
    if ((rc = cod_launch_gather_rows(c, H, a_rows, n_dev, R, c->D_in, c->hc, st)) != COD_OK) return rc;
    H = c->hc;
  }
  GemmArgs g{};
  g.A = H; g.lda = c->D_in; g.a_rows = nullptr; g.n_rows_dev = n_dev; g.rows_gate = dense_base; g.n_rows = R; g.K = c->D_in;
  g.seg[0] = {c->w.fc, c->D, c->wt.fc}; g.n_seg = 1; g.klass = COD_K_FC;
  // separate-projector variant, carry mode: F h and F_rej h of every row from one two-segment contraction,
  // the finish kernel keeps the one the row's status selects (the baseline keeps accepted rows only: F alone)
  const bool two = (f.flags & COD_F_REJ_PROJECTOR) && mode == COD_CARRY;
  if (two) { g.seg[1] = {c->w.fc_rej, c->D, c->wt.fc_rej}; g.n_seg = 2; }
  g.C = c->gemm_out; g.ldc = two ? 2 * c->D : c->D; g.splits = pick_splits(c, g.ldc, c->D_in, R);
  // More than 128 rows (tensor-bound): the contraction is grouped by row instead - the window is packed
  // accepted-first, rows [0, n_acc) meet F and rows [n_acc, R) meet F_rej in one launch, every row contracted
  // once. Up to 128 rows both matrices are streamed whole whatever the rows, and routing would save nothing.
  bool grouped = false;
  if (two && R > 128) {
    GemmArgs t = g;
    t.A = c->hc; t.ldc = c->D; t.group_split_dev = sp->acc_off + S;
    if (!c->force_simt && cod_gemm_tc2_supported(c, t)) {
      if ((rc = cod_launch_gather_grouped(c, H, sp, S, R, c->D_in, c->hc, c->perm, st)) != COD_OK) return rc;
      g = t;
      grouped = true;
    }
  }
  if ((rc = cod_launch_gemm(c, g, st)) != COD_OK) return rc;
  if ((rc = cod_launch_fc_finish(c, c->gemm_out, g.splits, R, n_dev, grouped ? c->perm : a_rows, sp->carry_slot, tap_z, st,
                                 g.ldc, dense_base, grouped ? 1 : 0)) != COD_OK)
    return rc;

  GemmArgs k{};
  k.A = c->z; k.lda = c->D; k.a_rows = nullptr; k.n_rows_dev = n_dev; k.rows_gate = dense_base; k.n_rows = R; k.K = c->D;
  k.seg[0] = {c->w.wk, f.n_layers * c->kvw, c->wt.wk};
  k.seg[1] = {c->w.wv, f.n_layers * c->kvw, c->wt.wv};
  k.n_seg = 2; k.klass = COD_K_KV;
  k.C = c->gemm_out; k.ldc = 2 * f.n_layers * c->kvw; k.splits = pick_splits(c, k.ldc, c->D, R);
  if ((rc = cod_launch_gemm(c, k, st)) != COD_OK) return rc;
  return cod_launch_kv_finish(c, c->gemm_out, k.splits, R, n_dev, a_rows, sp, J, dest, R, st, dense_base);
}

int cod_project_kv(cod_ctx* c, const void* H, const cod_split* split, int S, int mode, void* J,
                   cod_stream_t stream) {
  if (!c || !H || !J || split_has_null(split) || misaligned(H) || misaligned(J)) return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK || (mode != COD_CARRY && mode != COD_BASELINE)) return COD_ERR_INVALID_ARG;
  if (!c->has_weights) return COD_ERR_NO_WEIGHTS;
  c->pdl = true;
  return project_impl(c, H, split, S, mode, J, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

int cod_scatter_kv(cod_ctx* c, const void* J, const cod_split* split, int S, int mode, cod_state* st,
                   cod_stream_t stream) {
  if (!c || !J || split_has_null(split) || state_has_null(st) || misaligned(J) || misaligned(st->kv_pool) ||
      misaligned(st->carry_kv))
    return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK || (mode != COD_CARRY && mode != COD_BASELINE)) return COD_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  c->pdl = true;
  if (hist_missing(c, st)) return COD_ERR_INVALID_ARG;
  int rc = COD_OK;
  if (c->carry_base && (rc = cod_launch_carry_age(c, split, S, mode, st, s)) != COD_OK) return rc;
  if ((rc = cod_launch_scatter(c, J, split, S, mode, st, s)) != COD_OK) return rc;
  return cod_launch_update_lens(c, split, S, mode, st, s);
}

int cod_block_attn(cod_ctx* c, int layer, const void* q, const void* k_blk, const void* v_blk,
                   const cod_state* st, int S, int use_carry, void* out, float* carry_mass,
                   cod_stream_t stream) {
  if (!c || !q || !k_blk || !v_blk || !out || state_has_null(st)) return COD_ERR_INVALID_ARG;
  if (misaligned(q) || misaligned(k_blk) || misaligned(v_blk) || misaligned(out) || misaligned(st->kv_pool) ||
      misaligned(st->carry_kv))
    return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK || layer < 0 || layer >= c->cfg.n_layers) return COD_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  c->pdl = true;
  int rc = cod_launch_rope_blk_only(c, st->committed_len, S, s);
  if (rc != COD_OK) return rc;
  if ((rc = cod_launch_rope_qk(c, q, k_blk, st->committed_len, S, s)) != COD_OK) return rc;
  c->attn_order_stale = true;
  return cod_launch_attn(c, layer, c->q, c->kb, v_blk, st, S, use_carry ? 1 : 0, out, nullptr, carry_mass, s);
}

static int lm_head_impl(cod_ctx* c, int n_rows, cudaStream_t st) {
  GemmArgs g{};
  g.A = c->a; g.lda = c->D; g.n_rows = n_rows; g.K = c->D;
  g.seg[0] = {c->w.emb, c->cfg.vocab, c->emb_tiled}; g.n_seg = 1;
  g.splits = 1; g.amax = c->amax; g.klass = COD_K_LMHEAD;
  return cod_launch_gemm(c, g, st);
}

int cod_lm_head_argmax(cod_ctx* c, const float* x, int n_rows, int32_t* tok, float* top_logit,
                       cod_stream_t stream) {
  if (!c || !x || !tok || misaligned(x)) return COD_ERR_INVALID_ARG;
  if (n_rows < 1 || n_rows > c->R_max) return COD_ERR_INVALID_ARG;
  if (!c->has_weights) return COD_ERR_NO_WEIGHTS;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  c->pdl = true;
  int rc = cod_launch_resid_norm(c, nullptr, 0, n_rows, const_cast<float*>(x), c->w.g_final, nullptr, s);
  if (rc != COD_OK) return rc;
  if ((rc = lm_head_impl(c, n_rows, s)) != COD_OK) return rc;
  return cod_launch_finalize(c, n_rows, 1, nullptr, tok, nullptr, top_logit, s);
}

static int round_impl(cod_ctx* c, const int32_t* draft, const int32_t* target, const float* p_tok,
                      const float* q_tok, const float* u, const void* H, int S, int n_forced, int mode,
                      cod_state* st, cod_split* split_out, int32_t* next_draft, const cod_taps* taps,
                      cod_stream_t stream, float* q_next = nullptr, unsigned long long seed = 0, uint32_t step = 0) {
  const bool stochastic = p_tok != nullptr;
  if (!c || (!stochastic && !draft) || !target || !H || !next_draft || state_has_null(st)) return COD_ERR_INVALID_ARG;
  if (stochastic && (!q_tok || !u)) return COD_ERR_INVALID_ARG;
  if (misaligned(H) || misaligned(st->kv_pool) || misaligned(st->carry_kv)) return COD_ERR_INVALID_ARG;
  if (split_out && split_has_null(split_out)) return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK || n_forced < 0 || n_forced > 1) return COD_ERR_INVALID_ARG;
  if (mode != COD_CARRY && mode != COD_BASELINE) return COD_ERR_INVALID_ARG;
  if (!c->has_weights) return COD_ERR_NO_WEIGHTS;
  const cod_config& f = c->cfg;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const cod_split* sp = split_out ? split_out : &c->sp;
  const int R = S * f.block;
  const size_t es = esize(c);
  int rc;
  c->pdl = true;

  c->attn_order_stale = true;               // the lengths change below
  // part 1
  if ((rc = cod_launch_verify(c, draft, target, S, n_forced, st, sp, s, p_tok, q_tok, u)) != COD_OK) return rc;

  // retention beyond one round: the oldest round leaves U and the kept rows move to the front before
  // this round's rejected rows are written behind them
  if (hist_missing(c, st)) return COD_ERR_INVALID_ARG;
  if (c->carry_base && (rc = cod_launch_carry_age(c, sp, S, mode, st, s)) != COD_OK) return rc;

  // The first layer's embedding + Q/K/V chain of the NEXT block needs only the bonus tokens and the
  // position tables of part 1; the context projection (parts 2-3) needs only the row split. For
  // small rounds (a chain of short kernels) the former runs on a side stream next to the latter
  // and joins before the first attention; under stream capture the fork and join become graph edges.
  const bool fork = R <= c->side_rows && c->gemm_out2 != nullptr;
  cudaStream_t sq = fork ? c->side : s;                      // stream of the first layer's Q/K/V chain
  float* slab_q = fork ? c->gemm_out2 : c->gemm_out;
  if (fork) {
    if (cudaEventRecord(c->ev_fork, s) != cudaSuccess || cudaStreamWaitEvent(c->side, c->ev_fork, 0) != cudaSuccess)
      return COD_ERR_CUDA;
  } else {
    // parts 2-3 first, on the one stream
    if ((rc = project_impl(c, H, sp, S, mode, nullptr, st, taps ? taps->z : nullptr, s)) != COD_OK) return rc;
  }

  // the next block: [bonus, MASK, ...] through every drafter layer (the embedding kernel also
  // performs part 3's length update: nothing before the first attention reads the lengths)
  if ((rc = cod_launch_embed_norm(c, sp->bonus, S, sq, sp, mode, st)) != COD_OK) return rc;
  for (int l = 0; l < f.n_layers; ++l) {
    cudaStream_t sl = l == 0 ? sq : s;
    GemmArgs g{};
    g.A = c->a; g.lda = c->D; g.n_rows = R; g.K = c->D;
    auto tiled = [&](const char* base, int N, int K) -> const void* { return base ? base + l * cod_retile_bytes(N, K) : nullptr; };
    g.seg[0] = {static_cast<const char*>(c->w.wq) + es * l * c->qw * c->D, c->qw, tiled(c->wt.wq, c->qw, c->D)};
    g.seg[1] = {static_cast<const char*>(c->w.wk) + es * l * c->kvw * c->D, c->kvw, tiled(c->wt.wk, c->kvw, c->D)};
    g.seg[2] = {static_cast<const char*>(c->w.wv) + es * l * c->kvw * c->D, c->kvw, tiled(c->wt.wv, c->kvw, c->D)};
    g.n_seg = 3; g.klass = COD_K_QKV;
    g.C = l == 0 ? slab_q : c->gemm_out; g.ldc = c->qw + 2 * c->kvw; g.splits = pick_splits(c, g.ldc, c->D, R);
    if ((rc = cod_launch_gemm(c, g, sl)) != COD_OK) return rc;
    if ((rc = cod_launch_qkv_finish(c, g.C, g.splits, R, l, sl)) != COD_OK) return rc;
    if (l == 0 && fork) {
      // parts 2-3 on the caller's stream meanwhile, then the join
      if ((rc = project_impl(c, H, sp, S, mode, nullptr, st, taps ? taps->z : nullptr, s)) != COD_OK) return rc;
      if (cudaEventRecord(c->ev_join, c->side) != cudaSuccess || cudaStreamWaitEvent(s, c->ev_join, 0) != cudaSuccess)
        return COD_ERR_CUDA;
    }

    float* tap_o = (taps && taps->attn_out) ? taps->attn_out + static_cast<size_t>(l) * R * c->qw : nullptr;
    float* tap_m = (taps && taps->carry_mass) ? taps->carry_mass + static_cast<size_t>(l) * R * f.n_q_heads : nullptr;
    // after the join the first attention's stream predecessor is the context projection, which writes the pool,
    // the carry slots and (through the other branch) the lengths: that launch must not run ahead of it
    c->attn_run_ahead = !(l == 0 && fork);
    rc = cod_launch_attn(c, l, c->q, c->kb, c->vb, st, S, mode == COD_CARRY ? 1 : 0, c->o, tap_o, tap_m, s);
    c->attn_run_ahead = true;
    if (rc != COD_OK) return rc;

    GemmArgs o{};
    o.A = c->o; o.lda = c->qw; o.n_rows = R; o.K = c->qw;
    o.seg[0] = {static_cast<const char*>(c->w.wo) + es * l * c->D * c->qw, c->D, tiled(c->wt.wo, c->D, c->qw)};
    o.n_seg = 1; o.klass = COD_K_OPROJ;
    o.C = c->gemm_out; o.ldc = c->D; o.splits = pick_splits(c, c->D, c->qw, R);
    if ((rc = cod_launch_gemm(c, o, s)) != COD_OK) return rc;
    const bool last = l + 1 == f.n_layers;
    const void* gain = last ? c->w.g_final : static_cast<const char*>(c->w.g_attn) + es * (l + 1) * c->D;
    if (f.d_ff == 0) {
      if ((rc = cod_launch_resid_norm(c, c->gemm_out, o.splits, R, c->x, gain,
                                      (last && taps) ? taps->x_final : nullptr, s)) != COD_OK)
        return rc;
      continue;
    }
    // the gated MLP of the complete layer: b = N(x) g_mlp; x += W_down( silu(W_gate b) * (W_up b) )
    const void* g_mlp = static_cast<const char*>(c->w.g_mlp) + es * l * c->D;
    if ((rc = cod_launch_resid_norm(c, c->gemm_out, o.splits, R, c->x, g_mlp, nullptr, s)) != COD_OK) return rc;
    GemmArgs gu{};
    gu.A = c->a; gu.lda = c->D; gu.n_rows = R; gu.K = c->D;
    gu.seg[0] = {static_cast<const char*>(c->w.w_gate) + es * l * f.d_ff * c->D, f.d_ff, tiled(c->wt.w_gate, f.d_ff, c->D)};
    gu.seg[1] = {static_cast<const char*>(c->w.w_up) + es * l * f.d_ff * c->D, f.d_ff, tiled(c->wt.w_up, f.d_ff, c->D)};
    gu.n_seg = 2; gu.klass = COD_K_MLP;
    gu.C = c->gemm_out; gu.ldc = 2 * f.d_ff; gu.splits = pick_splits(c, gu.ldc, c->D, R);
    if ((rc = cod_launch_gemm(c, gu, s)) != COD_OK) return rc;
    if ((rc = cod_launch_swiglu_finish(c, c->gemm_out, gu.splits, R, s)) != COD_OK) return rc;
    GemmArgs dn{};
    dn.A = c->hmid; dn.lda = f.d_ff; dn.n_rows = R; dn.K = f.d_ff;
    dn.seg[0] = {static_cast<const char*>(c->w.w_down) + es * l * c->D * f.d_ff, c->D, tiled(c->wt.w_down, c->D, f.d_ff)};
    dn.n_seg = 1; dn.klass = COD_K_MLP;
    dn.C = c->gemm_out; dn.ldc = c->D; dn.splits = pick_splits(c, c->D, f.d_ff, R);
    if ((rc = cod_launch_gemm(c, dn, s)) != COD_OK) return rc;
    if ((rc = cod_launch_resid_norm(c, c->gemm_out, dn.splits, R, c->x, gain,
                                    (last && taps) ? taps->x_final : nullptr, s)) != COD_OK)
      return rc;
  }
  // part 5
  if (q_next != nullptr) {                      // temperature 1: the block is drawn, with its proposal probabilities
    GemmArgs g{};
    g.A = c->a; g.lda = c->D; g.n_rows = R; g.K = c->D;
    g.seg[0] = {c->w.emb, f.vocab, c->emb_tiled}; g.n_seg = 1;
    g.splits = 1; g.amax = c->amax; g.klass = COD_K_LMHEAD;
    g.lse_part = c->lse_part; g.sample_state = cod_sample_state(seed, step);
    if (c->force_simt || !(cod_gemm_tc2_supported(c, g) || cod_gemm_tc_supported(c, g))) return COD_ERR_UNSUPPORTED;
    if ((rc = cod_launch_gemm(c, g, s)) != COD_OK) return rc;
    return cod_launch_finalize_sample(c, R, g.sample_state, c->tok, q_next, nullptr, s, sp->bonus, next_draft);
  }
  if ((rc = lm_head_impl(c, R, s)) != COD_OK) return rc;
  return cod_launch_finalize(c, R, f.block, sp->bonus, c->tok, next_draft, taps ? taps->top_logit : nullptr, s);
}

int cod_lm_head_sample(cod_ctx* c, const float* x, int n_rows, unsigned long long seed, uint32_t step,
                       int32_t* tok, float* q_tok, float* lse, cod_stream_t stream) {
  if (!c || !x || !tok || misaligned(x)) return COD_ERR_INVALID_ARG;
  if (n_rows < 1 || n_rows > c->R_max) return COD_ERR_INVALID_ARG;
  if (!c->has_weights) return COD_ERR_NO_WEIGHTS;
  GemmArgs g{};
  g.A = c->a; g.lda = c->D; g.n_rows = n_rows; g.K = c->D;
  g.seg[0] = {c->w.emb, c->cfg.vocab, c->emb_tiled}; g.n_seg = 1;
  g.splits = 1; g.amax = c->amax; g.klass = COD_K_LMHEAD;
  g.lse_part = c->lse_part; g.sample_state = cod_sample_state(seed, step);
  if (c->force_simt || !(cod_gemm_tc2_supported(c, g) || cod_gemm_tc_supported(c, g))) return COD_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  c->pdl = true;
  int rc = cod_launch_resid_norm(c, nullptr, 0, n_rows, const_cast<float*>(x), c->w.g_final, nullptr, s);
  if (rc != COD_OK) return rc;
  if ((rc = cod_launch_gemm(c, g, s)) != COD_OK) return rc;
  return cod_launch_finalize_sample(c, n_rows, g.sample_state, tok, q_tok, lse, s);
}

int cod_lm_head_rank(cod_ctx* c, const float* x, int n_rows, const int32_t* ref_tok, int32_t* rank,
                     float* ref_logit, cod_stream_t stream) {
  if (!c || !x || !ref_tok || !rank || misaligned(x)) return COD_ERR_INVALID_ARG;
  if (n_rows < 1 || n_rows > c->R_max) return COD_ERR_INVALID_ARG;
  if (!c->has_weights) return COD_ERR_NO_WEIGHTS;
  GemmArgs g{};
  g.A = c->a; g.lda = c->D; g.n_rows = n_rows; g.K = c->D;
  g.seg[0] = {c->w.emb, c->cfg.vocab, c->emb_tiled}; g.n_seg = 1;
  g.splits = 1; g.klass = COD_K_LMHEAD;
  g.rank_ref = ref_logit ? ref_logit : reinterpret_cast<float*>(c->lse_part);   // scratch of the sampling head otherwise
  g.rank_tok = c->tok;
  g.rank_out = reinterpret_cast<unsigned int*>(rank);
  if (c->force_simt || !cod_gemm_tc_supported(c, g)) return COD_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  c->pdl = true;
  int rc = cod_launch_resid_norm(c, nullptr, 0, n_rows, const_cast<float*>(x), c->w.g_final, nullptr, s);
  if (rc != COD_OK) return rc;
  if ((rc = cod_launch_rank_ref(c, n_rows, ref_tok, const_cast<float*>(g.rank_ref), c->tok, rank, s)) != COD_OK) return rc;
  ProfScope prof(c, COD_K_LMHEAD, s);
  return cod_launch_gemm_tc(c, g, s);
}

int cod_draft_round(cod_ctx* c, const int32_t* draft, const int32_t* target, const void* H, int S,
                    int n_forced, int mode, cod_state* st, cod_split* split_out, int32_t* next_draft,
                    const cod_taps* taps, cod_stream_t stream) {
  if (!draft) return COD_ERR_INVALID_ARG;
  return round_impl(c, draft, target, nullptr, nullptr, nullptr, H, S, n_forced, mode, st, split_out, next_draft, taps, stream);
}

int cod_draft_round_stochastic(cod_ctx* c, const int32_t* target, const float* p_tok, const float* q_tok,
                               const float* u, const void* H, int S, int n_forced, int mode, cod_state* st,
                               cod_split* split_out, int32_t* next_draft, const cod_taps* taps,
                               float* q_next, unsigned long long seed, uint32_t step, cod_stream_t stream) {
  if (!p_tok || !q_tok || !u) return COD_ERR_INVALID_ARG;
  return round_impl(c, nullptr, target, p_tok, q_tok, u, H, S, n_forced, mode, st, split_out, next_draft, taps, stream,
                    q_next, seed, step);
}

int cod_reconvergence_count(cod_ctx* c, const int32_t* z, const int32_t* y, const int32_t* len, int S,
                            int32_t* R, cod_stream_t stream) {
  if (!c || !z || !y || !len || !R) return COD_ERR_INVALID_ARG;
  if (check_S(c, S) != COD_OK) return COD_ERR_INVALID_ARG;
  c->pdl = true;
  return cod_launch_reconvergence(c, z, y, len, S, R, static_cast<cudaStream_t>(stream));
}

int cod_poll_status(cod_ctx* c, uint32_t* dev_flags, int clear, cod_stream_t stream) {
  if (!c || !dev_flags) return COD_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(dev_flags, c->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess) return COD_ERR_CUDA;
  if (clear && cudaMemsetAsync(c->status, 0, sizeof(uint32_t), s) != cudaSuccess) return COD_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return COD_ERR_CUDA;
  return COD_OK;
}

int cod_set_wait_limit(cod_ctx* c, long long sm_cycles) {
  if (!c) return COD_ERR_INVALID_ARG;
  c->wait_limit = sm_cycles > 0 ? sm_cycles : 0;
  return COD_OK;
}

int cod_selftest_expire_wait(cod_ctx* c, int on) {
  if (!c) return COD_ERR_INVALID_ARG;
  c->selftest_skip_copies = on ? 1 : 0;
  return COD_OK;
}

int cod_profile_enable(cod_ctx* c, uint32_t class_mask) {
  if (!c) return COD_ERR_INVALID_ARG;
  c->prof_mask = class_mask & ((1u << COD_K_CLASSES) - 1u);
  c->prof_n = 0;
  return COD_OK;
}

int cod_profile_read(cod_ctx* c, int kernel_class, float* total_ms, int32_t* launches) {
  if (!c || !total_ms || !launches || kernel_class < 0 || kernel_class >= COD_K_CLASSES) return COD_ERR_INVALID_ARG;
  float tot = 0.f;
  int n = 0;
  for (int i = 0; i < c->prof_n; ++i) {
    if (c->prof_class[i] != kernel_class) continue;
    if (cudaEventSynchronize(c->prof_ev[2 * i + 1]) != cudaSuccess) return COD_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]) != cudaSuccess) return COD_ERR_CUDA;
    tot += ms;
    ++n;
  }
  *total_ms = tot;
  *launches = n;
  return COD_OK;
}

int64_t cod_launch_count(const cod_ctx* c) { return c ? c->launches : 0; }
int64_t cod_workspace_bytes(const cod_ctx* c) { return c ? static_cast<int64_t>(c->ws_bytes) : 0; }

const char* cod_error_string(int status) {
  switch (status) {
    case COD_OK: return "ok";
    case COD_ERR_INVALID_ARG: return "invalid argument";
    case COD_ERR_UNSUPPORTED: return "unsupported shape or flag";
    case COD_ERR_CUDA: return "CUDA runtime error";
    case COD_ERR_NO_WEIGHTS: return "weights not set";
    case COD_ERR_ALLOC: return "workspace allocation failed";
    case COD_ERR_TOO_LARGE: return "size exceeds a fixed capacity of this entry point";
    default: return "unknown status";
  }
}

}  // extern "C"
