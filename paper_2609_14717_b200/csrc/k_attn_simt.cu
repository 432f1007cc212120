// Part 4, general-shape path: split-KV block attention over [C_l; U_l; block] with plain FMA
// arithmetic and warp-shuffle softmax reductions (Section 2 "Preliminaries"; Algorithm 1 "the
// next draft reads ctx_l"). Used for float32 storage and for head sizes / block sizes the
// tensor-core kernel does not cover.
//
// Keys are addressed by one virtual index t: [0, L) committed rows through the page table,
// [L, L+c) the carried rows, [L+c, L+c+W) the block's own rows. A CTA owns one (sequence,
// KV head, split of split_len keys); the W * (n_q/n_kv) query rows that share the KV head are
// processed together so each K/V byte is read once per sequence. Split boundaries depend on
// the lengths only, so results do not depend on scheduling.
#include "cod_internal.cuh"

namespace {

constexpr int CH = 32;        // keys per chunk (one per lane)
constexpr int NWARP = 8;

template <typename T, int HD, int GPW>
__global__ void __launch_bounds__(NWARP * 32)
k_attn_split(const T* __restrict__ q, const T* __restrict__ kb, const T* __restrict__ vb,
             const T* __restrict__ pool, const T* __restrict__ carry, const int* __restrict__ block_table,
             const int* __restrict__ committed_len, const int* __restrict__ carry_len, int use_carry,
             int layer, int W, int rep, int n_kv, int page, int max_pages, int n_pages, int max_batch,
             int split_len, int max_splits, float* __restrict__ part_o, float* __restrict__ part_ml,
             uint32_t* status, int cap /* rows of a carry slot */) {
  cod_pdl_prologue();
  extern __shared__ float smem[];
  const int M = W * rep;
  float* Qs = smem;                       // [M][HD]   (pre-scaled by 1/sqrt(hd))
  float* Ks = Qs + M * HD;                // [CH][HD+1]
  float* Vs = Ks + CH * (HD + 1);         // [CH][HD]

  const int k = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
  int L = committed_len[s];
  int c = use_carry ? carry_len[s] : 0;
  uint32_t flags = 0;
  if (L < 0 || L > max_pages * page) { flags |= COD_DEV_BAD_LEN; L = max(0, min(L, max_pages * page)); }
  if (c < 0 || c > cap) { flags |= COD_DEV_BAD_LEN; c = max(0, min(c, cap)); }
  const int T_total = L + c + W;
  const int t0 = k * split_len;
  if (t0 >= T_total) return;
  const int t1 = min(T_total, t0 + split_len);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qw = n_kv * rep * HD, kvw = n_kv * HD;
  const float scale = rsqrtf(static_cast<float>(HD));
  for (int idx = tid; idx < M * HD; idx += blockDim.x) {
    const int mrow = idx / HD, d = idx - mrow * HD;
    const int i = mrow / rep, gg = mrow - i * rep;
    Qs[idx] = cod_ld(q + static_cast<size_t>(s * W + i) * qw + (h * rep + gg) * HD + d) * scale;
  }

  constexpr int DD = HD / 32;
  float o[GPW][4][DD];
  float m_run[GPW][4], l_run[GPW][4], lc_run[GPW][4];
#pragma unroll
  for (int g = 0; g < GPW; ++g)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      m_run[g][r] = -INFINITY; l_run[g][r] = 0.f; lc_run[g][r] = 0.f;
#pragma unroll
      for (int dd = 0; dd < DD; ++dd) o[g][r][dd] = 0.f;
    }

  for (int t = t0; t < t1; t += CH) {
    const int n_valid = min(CH, t1 - t);
    __syncthreads();
    for (int idx = tid; idx < CH * (HD / 4); idx += blockDim.x) {
      const int key = idx / (HD / 4), d4 = (idx - key * (HD / 4)) * 4;
      float4 kv4 = make_float4(0.f, 0.f, 0.f, 0.f), vv4 = kv4;
      if (key < n_valid) {
        const int tt = t + key;
        const T *kp, *vp;
        if (tt < L) {
          int pg = block_table[s * max_pages + tt / page];
          if (pg < 0 || pg >= n_pages) { flags |= COD_DEV_BAD_PAGE; pg = 0; }
          kp = pool + ((((static_cast<size_t>(layer) * n_pages + pg) * n_kv + h) * 2) * page + tt % page) * HD;
          vp = kp + static_cast<size_t>(page) * HD;
        } else if (tt < L + c) {
          kp = carry + ((((static_cast<size_t>(layer) * max_batch + s) * n_kv + h) * 2) * cap + (tt - L)) * HD;
          vp = kp + static_cast<size_t>(cap) * HD;
        } else {
          const int i = tt - L - c;
          kp = kb + static_cast<size_t>(s * W + i) * kvw + h * HD;
          vp = vb + static_cast<size_t>(s * W + i) * kvw + h * HD;
        }
        kv4 = cod_ld4(kp + d4);
        vv4 = cod_ld4(vp + d4);
      }
      float* kd = Ks + key * (HD + 1) + d4;
      kd[0] = kv4.x; kd[1] = kv4.y; kd[2] = kv4.z; kd[3] = kv4.w;
      *reinterpret_cast<float4*>(Vs + key * HD + d4) = vv4;
    }
    __syncthreads();

    const bool valid = lane < n_valid;
    const bool is_carry = valid && (t + lane >= L) && (t + lane < L + c);
#pragma unroll
    for (int g = 0; g < GPW; ++g) {
      const int row0 = (warp + g * NWARP) * 4;
      if (row0 >= M) continue;
      float sc[4] = {0.f, 0.f, 0.f, 0.f};
      const float* kr = Ks + lane * (HD + 1);
#pragma unroll 8
      for (int d = 0; d < HD; ++d) {
        const float kvv = kr[d];
#pragma unroll
        for (int r = 0; r < 4; ++r) sc[r] = fmaf(Qs[min(row0 + r, M - 1) * HD + d], kvv, sc[r]);
      }
      float p[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const float sv = valid ? sc[r] : -INFINITY;
        const float m_new = fmaxf(m_run[g][r], cod_warp_max(sv));
        p[r] = valid ? __expf(sv - m_new) : 0.f;
        const float corr = __expf(m_run[g][r] - m_new);     // exp(-inf) = 0 on the first chunk
        l_run[g][r] = l_run[g][r] * corr + cod_warp_sum(p[r]);
        lc_run[g][r] = lc_run[g][r] * corr + cod_warp_sum(is_carry ? p[r] : 0.f);
        m_run[g][r] = m_new;
#pragma unroll
        for (int dd = 0; dd < DD; ++dd) o[g][r][dd] *= corr;
      }
      for (int j = 0; j < n_valid; ++j) {
        float vv[DD];
#pragma unroll
        for (int dd = 0; dd < DD; ++dd) vv[dd] = Vs[j * HD + lane + 32 * dd];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const float pj = __shfl_sync(0xffffffffu, p[r], j);
#pragma unroll
          for (int dd = 0; dd < DD; ++dd) o[g][r][dd] = fmaf(pj, vv[dd], o[g][r][dd]);
        }
      }
    }
  }

  const size_t base = ((static_cast<size_t>(s) * n_kv + h) * max_splits + k) * M;
#pragma unroll
  for (int g = 0; g < GPW; ++g)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = (warp + g * NWARP) * 4 + r;
      if (row >= M) continue;
#pragma unroll
      for (int dd = 0; dd < DD; ++dd) part_o[(base + row) * HD + lane + 32 * dd] = o[g][r][dd];
      if (lane == 0) {
        float* ml = part_ml + (base + row) * 4;
        ml[0] = m_run[g][r]; ml[1] = l_run[g][r]; ml[2] = lc_run[g][r];
      }
    }
  if (flags) atomicOr(status, flags);
}

// Merges the splits of one (row, query head) by log-sum-exp weights; one warp each.
template <typename T, int HD>
__global__ void k_attn_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                               const int* __restrict__ committed_len, const int* __restrict__ carry_len,
                               int use_carry, int S, int W, int rep, int n_kv, int page, int max_pages,
                               int split_len, int max_splits, T* __restrict__ out, float* __restrict__ tap,
                               float* __restrict__ mass, int cap) {
  cod_pdl_prologue();
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // (s, i, g)
  const int n_q = n_kv * rep;
  if (item >= S * W * n_q) return;
  const int g = item % n_q, i = (item / n_q) % W, s = item / (n_q * W);
  const int h = g / rep, mrow = i * rep + (g - h * rep), M = W * rep;
  const int L = max(0, min(committed_len[s], max_pages * page));
  const int c = use_carry ? max(0, min(carry_len[s], cap)) : 0;
  const int n_splits = (L + c + W + split_len - 1) / split_len;
  const size_t base = (static_cast<size_t>(s) * n_kv + h) * max_splits;

  float mg = -INFINITY;
  for (int k = 0; k < n_splits; ++k) mg = fmaxf(mg, part_ml[((base + k) * M + mrow) * 4]);
  constexpr int DD = HD / 32;
  float acc[DD] = {}, l = 0.f, lc = 0.f;
  for (int k = 0; k < n_splits; ++k) {
    const float* ml = part_ml + ((base + k) * M + mrow) * 4;
    const float w = __expf(ml[0] - mg);
    l = fmaf(w, ml[1], l);
    lc = fmaf(w, ml[2], lc);
    const float* po = part_o + ((base + k) * M + mrow) * HD;
#pragma unroll
    for (int dd = 0; dd < DD; ++dd) acc[dd] = fmaf(w, po[lane + 32 * dd], acc[dd]);
  }
  const float inv = 1.f / l;
  const size_t ob = static_cast<size_t>(item) * HD;      // [s][i][g][d]
#pragma unroll
  for (int dd = 0; dd < DD; ++dd) {
    const float v = acc[dd] * inv;
    cod_st(out + ob + lane + 32 * dd, v);
    if (tap) tap[ob + lane + 32 * dd] = v;
  }
  if (mass && lane == 0) mass[item] = lc * inv;
}

template <typename T, int HD, int GPW>
int launch_split(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb, const cod_state* stt,
                 int S, int use_carry, cudaStream_t st) {
  const cod_config& f = c->cfg;
  const int rep = f.n_q_heads / f.n_kv_heads, M = f.block * rep;
  const size_t smem = (static_cast<size_t>(M) * HD + CH * (HD + 1) + CH * HD) * sizeof(float);
  auto kern = k_attn_split<T, HD, GPW>;
  if (smem > 48 * 1024) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
      return COD_ERR_CUDA;
  }
  dim3 grid(c->max_splits, f.n_kv_heads, S);
  cod_launch_pdl(c, kern, grid, NWARP * 32, smem, st, static_cast<const T*>(q), static_cast<const T*>(kb), static_cast<const T*>(vb),
                                       static_cast<const T*>(stt->kv_pool), static_cast<const T*>(stt->carry_kv),
                                       stt->block_table, stt->committed_len, stt->carry_len, use_carry, layer, f.block,
                                       rep, f.n_kv_heads, f.page_size, f.max_pages_per_seq, f.n_pages, f.max_batch,
                                       c->split_len, c->max_splits, c->attn_o, c->attn_ml, c->status, c->carry_cap);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

template <typename T, int HD>
int launch_all(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb, const cod_state* stt, int S,
               int use_carry, void* out, float* tap, float* mass, cudaStream_t st) {
  const cod_config& f = c->cfg;
  const int rep = f.n_q_heads / f.n_kv_heads, M = f.block * rep;
  int rc;
  if (M <= 32) rc = launch_split<T, HD, 1>(c, layer, q, kb, vb, stt, S, use_carry, st);
  else if (M <= 64) rc = launch_split<T, HD, 2>(c, layer, q, kb, vb, stt, S, use_carry, st);
  else if (M <= 128) rc = launch_split<T, HD, 4>(c, layer, q, kb, vb, stt, S, use_carry, st);
  else return COD_ERR_UNSUPPORTED;
  if (rc != COD_OK) return rc;
  const int items = S * f.block * f.n_q_heads;
  cod_launch_pdl(c, k_attn_combine<T, HD>, (items + 3) / 4, 128, 0, st, c->attn_o, c->attn_ml, stt->committed_len, stt->carry_len,
                                                         use_carry, S, f.block, rep, f.n_kv_heads, f.page_size,
                                                         f.max_pages_per_seq, c->split_len, c->max_splits,
                                                         static_cast<T*>(out), tap, mass, c->carry_cap);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

}  // namespace

// q / kb: already rotated. out [S, W, n_q, hd]; tap (nullable) the same values in float.
int cod_launch_attn_simt(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb,
                         const cod_state* stt, int S, int use_carry, void* out, float* tap, float* mass,
                         cudaStream_t st) {
  const int hd = c->cfg.head_dim;
  if (c->cfg.dtype == COD_BF16) {
    if (hd == 128) return launch_all<__nv_bfloat16, 128>(c, layer, q, kb, vb, stt, S, use_carry, out, tap, mass, st);
    if (hd == 64) return launch_all<__nv_bfloat16, 64>(c, layer, q, kb, vb, stt, S, use_carry, out, tap, mass, st);
  } else {
    if (hd == 128) return launch_all<float, 128>(c, layer, q, kb, vb, stt, S, use_carry, out, tap, mass, st);
    if (hd == 64) return launch_all<float, 64>(c, layer, q, kb, vb, stt, S, use_carry, out, tap, mass, st);
  }
  return COD_ERR_UNSUPPORTED;
}
