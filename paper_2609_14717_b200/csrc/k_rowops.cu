// Row-wise kernels between the contractions: split-K reduction, E_carry on rejected rows,
// RMS norms, RoPE, the K/V scatter, the embedding gather and the argmax read-out.
#include "cod_internal.cuh"

namespace {

// Row kernels keep a row in registers as NV float4 slots per thread (D <= 4 * NV * blockDim.x):
// one slot with up to 1024 threads for rows of up to 4096 elements, eight slots beyond.
constexpr int ROW_WIDE_NV = 8;

__device__ __forceinline__ void cod_st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void cod_st4(__nv_bfloat16* p, float4 v) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<const uint32_t*>(&a);
  u.y = *reinterpret_cast<const uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
__device__ __forceinline__ float4 f4_add(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }
__device__ __forceinline__ float f4_ss(float4 a) { return a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w; }

// Sum over the `group` consecutive lanes (a power of two <= 32) a head's threads occupy.
__device__ __forceinline__ float group_sum(float v, int group) {
  for (int o = group >> 1; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float4 f4_scale_gain(float4 v, float s, float4 g) {
  return make_float4(v.x * s * g.x, v.y * s * g.y, v.z * s * g.z, v.w * s * g.w);
}

__device__ __forceinline__ int valid_rows(const int* n_rows_dev, int n_rows) {
  return n_rows_dev ? min(*n_rows_dev, n_rows) : n_rows;
}

// ------------------------------------------------------------------ F(E_carry) = fc . e_carry
// F is linear and bias-free, so F(h + E_carry) = F(h) + F(E_carry) (Eq. 2; Algorithm 1, right
// column, step 2): the embedding can be added after the contraction, before the norm.
template <typename T>
__global__ void k_fcE(const T* __restrict__ fc, const T* __restrict__ e, int D_in, float* __restrict__ out) {
  cod_pdl_prologue();
  __shared__ float red[33];
  const int n = blockIdx.x;
  float acc = 0.f;
  for (int k = threadIdx.x; k < D_in; k += blockDim.x) acc = fmaf(cod_ld(fc + static_cast<size_t>(n) * D_in + k), cod_ld(e + k), acc);
  acc = cod_block_sum(acc, red);
  if (threadIdx.x == 0) out[n] = acc;
}

// ------------------------------------------------------------------ row compaction (baseline mode)
// dst[i] = src[rows[i]] for i < *n_dev: the accepted rows of H packed densely, so the baseline
// column of Algorithm 1 ("collect accepted states") runs the same dense contractions on fewer rows.
template <typename T>
__global__ void k_gather_rows(const T* __restrict__ src, const int* __restrict__ rows, const int* __restrict__ n_dev,
                              int width, T* __restrict__ dst) {
  cod_pdl_prologue();
  const int i = blockIdx.x;
  if (i >= *n_dev) return;
  const int row = rows[i];
  constexpr int VEC = 16 / sizeof(T);
  const uint4* s4 = reinterpret_cast<const uint4*>(src + static_cast<size_t>(row) * width);
  uint4* d4 = reinterpret_cast<uint4*>(dst + static_cast<size_t>(i) * width);
  for (int e = threadIdx.x; e < width / VEC; e += blockDim.x) d4[e] = s4[e];
}

// dst[i] = src[perm[i]] with perm = the accepted rows (in order), then the rejected rows (in order): the window
// grouped by row status, so that a contraction can meet each group with its own weights.
template <typename T>
__global__ void k_gather_grouped(const T* __restrict__ src, const int* __restrict__ acc_rows, const int* __restrict__ n_acc_dev,
                                 const int* __restrict__ rej_rows, int width, T* __restrict__ dst, int* __restrict__ perm) {
  cod_pdl_prologue();
  const int i = blockIdx.x, n_acc = *n_acc_dev;
  const int row = i < n_acc ? acc_rows[i] : rej_rows[i - n_acc];
  if (threadIdx.x == 0) perm[i] = row;
  constexpr int VEC = 16 / sizeof(T);
  const uint4* s4 = reinterpret_cast<const uint4*>(src + static_cast<size_t>(row) * width);
  uint4* d4 = reinterpret_cast<uint4*>(dst + static_cast<size_t>(i) * width);
  for (int e = threadIdx.x; e < width / VEC; e += blockDim.x) d4[e] = s4[e];
}

// ------------------------------------------------------------------ fc finish
// z[row] = N_h( sum_splits part[i] + [row rejected] F(E_carry) )   (one block per kept row)
template <typename T, int NV>
__global__ void __launch_bounds__(1024) k_fc_finish(const float* __restrict__ part, int splits, int n_rows, const int* n_rows_dev,
                            const int* __restrict__ a_rows, const int* __restrict__ carry_slot,
                            const float* __restrict__ fcE, const T* __restrict__ gain, int D, float eps,
                            int do_norm, T* __restrict__ z, int z_compact, float* __restrict__ tap, int ldp, int dense_base) {
  cod_pdl_prologue();
  __shared__ float red[33];
  const int i = blockIdx.x;
  // dense_base: the baseline drafter on ALL window rows (the contraction ran on every row because extra token
  // columns are free while it streams weights); only accepted rows exist for it, and none if none was accepted
  if (i >= (dense_base ? (*n_rows_dev > 0 ? n_rows : 0) : valid_rows(n_rows_dev, n_rows))) return;
  const int row = a_rows ? a_rows[i] : i;
  const bool rej = carry_slot[row] >= 0;
  if (dense_base && rej) return;
  const int nv = D >> 2;
  float4 v[NV];
  float ss = 0.f;
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    v[t] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < nv && rej && fcE != nullptr) v[t] = *reinterpret_cast<const float4*>(fcE + 4 * j);
  }
  // ldp = D: one projection per row. ldp = 2 D: F h and F_rej h side by side, rejected rows take the second.
  const float* prow = part + static_cast<size_t>(i) * ldp + ((ldp > D && rej) ? D : 0);
  if (NV == 1) {
    // one slot per thread: every slab's load is requested before the first sum (same order of sums)
#pragma unroll
    for (int s = 0; s < COD_MAX_SPLITS; ++s)
      if (s < splits && static_cast<int>(threadIdx.x) < nv)
        v[0] = f4_add(v[0], *reinterpret_cast<const float4*>(prow + static_cast<size_t>(s) * n_rows * ldp + 4 * threadIdx.x));
  }
#pragma unroll 4
  for (int s = NV == 1 ? COD_MAX_SPLITS : 0; s < splits; ++s) {   // slots inside, four slabs unrolled: their loads are in flight together
#pragma unroll
    for (int t = 0; t < NV; ++t) {
      const int j = threadIdx.x + t * blockDim.x;
      if (j < nv) v[t] = f4_add(v[t], *reinterpret_cast<const float4*>(prow + static_cast<size_t>(s) * n_rows * ldp + 4 * j));
    }
  }
#pragma unroll
  for (int t = 0; t < NV; ++t) ss += f4_ss(v[t]);
  ss = cod_block_sum(ss, red);
  // the partial sums are dead: their lines leave L2 without a write-back (the block has met since their last read)
  if ((D & 31) == 0 && (ldp & 31) == 0 && gridDim.x > COD_DROP_MIN_ROWS) {
#pragma unroll
    for (int t = 0; t < NV; ++t) {
      const int j = threadIdx.x + t * blockDim.x;
      if (j < nv)
        for (int s = j & 7; s < splits; s += 8) cod_discard_line(prow + static_cast<size_t>(s) * n_rows * ldp + 4 * (j & ~7));
    }
  }
  const float scale = do_norm ? rsqrtf(ss / static_cast<float>(D) + eps) : 1.f;
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    if (j < nv) {
      float4 o = v[t];
      if (do_norm) {
        const float4 g = cod_ld4(gain + 4 * j);
        o = make_float4(o.x * scale * g.x, o.y * scale * g.y, o.z * scale * g.z, o.w * scale * g.w);
      }
      cod_st4(z + static_cast<size_t>(z_compact ? i : row) * D + 4 * j, o);
      if (tap) *reinterpret_cast<float4*>(tap + static_cast<size_t>(row) * D + 4 * j) = o;
    }
  }
}

// ------------------------------------------------------------------ K/V finish
// part: [splits][n_rows][2 * Ld * kvw]; columns [0, Ld*kvw) are K of every layer, the rest V.
// Rotates K at the row's position and writes either J[l][row][2][n_kv][hd] or straight to the
// row's destination (page slot if accepted, carry slot if rejected).
template <typename T>
__global__ void k_kv_finish(const float* __restrict__ part, int splits, int n_rows, const int* n_rows_dev,
                            const int* __restrict__ a_rows, const float* __restrict__ rope_win, int Ld,
                            int n_kv, int hd, T* __restrict__ J, int R_total,
                            const int* __restrict__ commit_slot, const int* __restrict__ carry_slot,
                            T* __restrict__ pool, T* __restrict__ carry, int page, int n_pages, int W,
                            int max_batch, int to_state, const T* __restrict__ g_k, float eps, int cap,
                            const int* __restrict__ carry_base, int dense_base) {
  cod_pdl_prologue();
  const int i = blockIdx.x, l = blockIdx.y;
  if (i >= (dense_base ? (*n_rows_dev > 0 ? n_rows : 0) : valid_rows(n_rows_dev, n_rows))) return;
  const int row = a_rows ? a_rows[i] : i;
  if (dense_base && carry_slot[row] >= 0) return;   // the baseline drafter keeps no rejected row
  const int kvw = n_kv * hd, half = hd >> 1, ldc = 2 * Ld * kvw;
  const float* cs = rope_win + static_cast<size_t>(row) * hd;

  T* dstK = nullptr;   // address of [h = 0][K][..][d = 0]; strides below
  size_t h_stride, kv_stride;
  if (!to_state) {
    dstK = J + ((static_cast<size_t>(l) * R_total + row) * 2) * kvw;
    h_stride = hd;
    kv_stride = kvw;
  } else {
    const int cslot = commit_slot[row], uslot = carry_slot[row];
    if (cslot >= 0) {
      const int pg = cslot / page, off = cslot - pg * page;
      dstK = pool + (((static_cast<size_t>(l) * n_pages + pg) * n_kv) * 2) * page * hd + static_cast<size_t>(off) * hd;
      h_stride = static_cast<size_t>(2) * page * hd;
      kv_stride = static_cast<size_t>(page) * hd;
    } else if (uslot >= 0 && carry) {
      // a carry slot holds cap = k * W rows; the new round's rows follow the carry_base[s] retained ones
      const int s = uslot / W, u = uslot - s * W + (carry_base ? carry_base[s] : 0);
      dstK = carry + (((static_cast<size_t>(l) * max_batch + s) * n_kv) * 2) * cap * hd + static_cast<size_t>(u) * hd;
      h_stride = static_cast<size_t>(2) * cap * hd;
      kv_stride = static_cast<size_t>(cap) * hd;
    } else {
      return;   // nowhere to go (position beyond the page table: already flagged)
    }
  }
  // hd / 8 threads per head: 4 consecutive elements of the lower half and their RoPE partners.
  // With the per-head key norm (g_k non-null, gains of layer l at g_k + l * hd) a head's threads
  // first share the key's sum of squares; whole warps stay in the loop for those shuffles.
  const int tph = half >> 2;
  for (int e0 = 0; e0 < n_kv * tph; e0 += blockDim.x) {
    const int e = e0 + threadIdx.x;
    const bool live = e < n_kv * tph;
    const int h = live ? e / tph : 0, j = live ? (e - h * tph) * 4 : 0;
    float4 k1 = make_float4(0.f, 0.f, 0.f, 0.f), k2 = k1, v1 = k1, v2 = k1;
    const float* p = part + static_cast<size_t>(i) * ldc + l * kvw + h * hd + j;
    const size_t slab = static_cast<size_t>(n_rows) * ldc;
    if (live) {
#pragma unroll 4
      for (int s = 0; s < splits; ++s) {
        k1 = f4_add(k1, *reinterpret_cast<const float4*>(p + s * slab));
        k2 = f4_add(k2, *reinterpret_cast<const float4*>(p + s * slab + half));
        v1 = f4_add(v1, *reinterpret_cast<const float4*>(p + s * slab + Ld * kvw));
        v2 = f4_add(v2, *reinterpret_cast<const float4*>(p + s * slab + Ld * kvw + half));
      }
    }
    if ((half & 31) == 0 && gridDim.x > COD_DROP_MIN_ROWS) {          // the partial sums are dead: dropped from L2, no write-back (see k_qkv_finish)
      __syncwarp();
      const int g8 = threadIdx.x & 7;                // the eight lanes share the drops
      if (live)
        for (int idx = g8; idx < 4 * splits; idx += 8)
          cod_discard_line(p - 4 * g8 + (idx >> 2) * slab + ((idx >> 1) & 1) * (Ld * kvw) + (idx & 1) * half);
    }
    if (g_k != nullptr) {
      const float ss = group_sum(f4_ss(k1) + f4_ss(k2), tph);
      const float sc = rsqrtf(ss / static_cast<float>(hd) + eps);
      if (live) {
        k1 = f4_scale_gain(k1, sc, cod_ld4(g_k + l * hd + j));
        k2 = f4_scale_gain(k2, sc, cod_ld4(g_k + l * hd + half + j));
      }
    }
    if (!live) continue;
    const float4 c = *reinterpret_cast<const float4*>(cs + j), sn = *reinterpret_cast<const float4*>(cs + half + j);
    T* kd = dstK + h * h_stride;
    cod_st4(kd + j, make_float4(k1.x * c.x - k2.x * sn.x, k1.y * c.y - k2.y * sn.y, k1.z * c.z - k2.z * sn.z, k1.w * c.w - k2.w * sn.w));
    cod_st4(kd + j + half, make_float4(k2.x * c.x + k1.x * sn.x, k2.y * c.y + k1.y * sn.y, k2.z * c.z + k1.z * sn.z, k2.w * c.w + k1.w * sn.w));
    cod_st4(kd + kv_stride + j, v1);
    cod_st4(kd + kv_stride + j + half, v2);
  }
}

// ------------------------------------------------------------------ scatter (unfused form)
// One block per (row, layer): copies the row's K and V (n_kv heads of hd elements each) from J
// to its page slot or carry slot with 128-bit accesses.
template <typename T>
__global__ void k_scatter_kv(const T* __restrict__ J, int R_total, int n_kv, int hd,
                             const int* __restrict__ commit_slot, const int* __restrict__ carry_slot,
                             T* __restrict__ pool, T* __restrict__ carry, int page, int n_pages, int W,
                             int max_batch, int use_carry, int cap, const int* __restrict__ carry_base) {
  cod_pdl_prologue();
  const int row = blockIdx.x, l = blockIdx.y;
  const int kvw = n_kv * hd;
  const int cslot = commit_slot[row], uslot = carry_slot[row];
  T* dst;
  size_t h_stride, kv_stride;
  if (cslot >= 0) {
    const int pg = cslot / page, off = cslot - pg * page;
    dst = pool + (((static_cast<size_t>(l) * n_pages + pg) * n_kv) * 2) * page * hd + static_cast<size_t>(off) * hd;
    h_stride = static_cast<size_t>(2) * page * hd;
    kv_stride = static_cast<size_t>(page) * hd;
  } else if (uslot >= 0 && use_carry) {
    const int s = uslot / W, u = uslot - s * W + (carry_base ? carry_base[s] : 0);
    dst = carry + (((static_cast<size_t>(l) * max_batch + s) * n_kv) * 2) * cap * hd + static_cast<size_t>(u) * hd;
    h_stride = static_cast<size_t>(2) * cap * hd;
    kv_stride = static_cast<size_t>(cap) * hd;
  } else {
    return;
  }
  constexpr int VEC = 16 / sizeof(T);
  const T* src = J + ((static_cast<size_t>(l) * R_total + row) * 2) * kvw;
  const int per_head = hd / VEC;
  for (int e = threadIdx.x; e < 2 * n_kv * per_head; e += blockDim.x) {
    const int kv = e / (n_kv * per_head), rem = e - kv * n_kv * per_head;
    const int h = rem / per_head, v = rem - h * per_head;
    const uint4 val = *reinterpret_cast<const uint4*>(src + static_cast<size_t>(kv) * kvw + h * hd + v * VEC);
    *reinterpret_cast<uint4*>(dst + h * h_stride + kv * kv_stride + v * VEC) = val;
  }
}

// committed_len[s] += m_s; carry_len[s] = kept rows + W - m_s (0 for the baseline drafter)
struct LensUpdate {
  const int* accept_len;      // null: no update
  int S, W, mode, max_tokens;
  int* committed_len;
  int* carry_len;
  uint32_t* status;
  const int* carry_base;
};
__device__ __forceinline__ void cod_update_lens_one(const LensUpdate& u, int s) {
  const int m = u.accept_len[s];
  const int L = u.committed_len[s] + m;
  if (L > u.max_tokens) atomicOr(u.status, COD_DEV_PAGE_OVERFLOW);
  u.committed_len[s] = L;
  u.carry_len[s] = u.mode == COD_CARRY ? (u.carry_base ? u.carry_base[s] : 0) + u.W - m : 0;
}
__global__ void k_update_lens(LensUpdate u) {
  cod_pdl_prologue();
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s < u.S) cod_update_lens_one(u, s);
}

// ------------------------------------------------------------------ carry retention (carry_rounds = k > 1)
// Per sequence: the oldest of the k retained rounds leaves U. hist[s][0..k) holds the segment lengths,
// oldest first (zeros at the start: empty rounds). base[s] = rows that stay; the history shifts and
// takes the new round's W - m. The baseline drafter keeps no U: history and base are cleared.
__global__ void k_carry_age_hist(const int* __restrict__ accept_len, const int* __restrict__ carry_len, int S, int W,
                                 int k, int mode, int* __restrict__ hist, int* __restrict__ base, int* __restrict__ drop) {
  cod_pdl_prologue();
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= S) return;
  int* h = hist + static_cast<size_t>(s) * k;
  if (mode != COD_CARRY) {
    for (int j = 0; j < k; ++j) h[j] = 0;
    base[s] = 0; drop[s] = 0;
    return;
  }
  int keep = 0;
  for (int j = 1; j < k; ++j) { keep += h[j]; h[j - 1] = h[j]; }
  h[k - 1] = W - accept_len[s];
  keep = max(0, min(keep, carry_len[s]));
  base[s] = keep;
  drop[s] = max(0, carry_len[s] - keep);
}
// Moves rows [drop, drop + keep) of every (layer, sequence, head, K|V) slot to the front. One block per
// slot; rows go one at a time in increasing order (destination below source), a barrier between the
// read and the write of a row.
template <typename T>
__global__ void k_carry_shift(T* __restrict__ carry, const int* __restrict__ base, const int* __restrict__ drop,
                              int max_batch, int n_kv, int cap, int hd) {
  cod_pdl_prologue();
  const int s = blockIdx.x, slot = blockIdx.y, l = blockIdx.z;          // slot = head * 2 + (K|V)
  const int keep = base[s], d = drop[s];
  if (d == 0 || keep == 0) return;
  T* p = carry + ((static_cast<size_t>(l) * max_batch + s) * n_kv * 2 + slot) * cap * hd;
  for (int i = 0; i < keep; ++i) {
    T v = T();
    if (threadIdx.x < hd) v = p[static_cast<size_t>(i + d) * hd + threadIdx.x];
    __syncthreads();
    if (threadIdx.x < hd) p[static_cast<size_t>(i) * hd + threadIdx.x] = v;
    __syncthreads();
  }
}

// ------------------------------------------------------------------ block input
// x = Emb[[bonus, MASK, ...]], a = N(x) * g_attn[0]; also clears the argmax keys.
template <typename T, int NV>
__global__ void __launch_bounds__(1024) k_embed_norm(const T* __restrict__ emb, const int* __restrict__ bonus, int W, int mask_id,
                             int vocab, const T* __restrict__ gain, int D, float eps, float* __restrict__ x,
                             T* __restrict__ a, unsigned long long* __restrict__ amax, LensUpdate lu) {
  cod_pdl_prologue();
  __shared__ float red[33];
  const int r = blockIdx.x, s = r / W, p = r - s * W;
  // inside a round this kernel also carries the length update of part 3 (one launch fewer on the
  // critical path; nothing between part 1 and the first attention reads the lengths)
  if (blockIdx.x == 0 && lu.accept_len != nullptr)
    for (int q = threadIdx.x; q < lu.S; q += blockDim.x) cod_update_lens_one(lu, q);
  int tok = p == 0 ? bonus[s] : mask_id;
  if (tok < 0 || tok >= vocab) tok = 0;
  const int nv = D >> 2;
  float4 v[NV];
  float ss = 0.f;
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    v[t] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < nv) {
      v[t] = cod_ld4(emb + static_cast<size_t>(tok) * D + 4 * j);
      *reinterpret_cast<float4*>(x + static_cast<size_t>(r) * D + 4 * j) = v[t];
      ss += f4_ss(v[t]);
    }
  }
  ss = cod_block_sum(ss, red);
  const float scale = rsqrtf(ss / static_cast<float>(D) + eps);
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    if (j < nv) {
      const float4 g = cod_ld4(gain + 4 * j);
      cod_st4(a + static_cast<size_t>(r) * D + 4 * j,
              make_float4(v[t].x * scale * g.x, v[t].y * scale * g.y, v[t].z * scale * g.z, v[t].w * scale * g.w));
    }
  }
  if (threadIdx.x == 0) amax[r] = 0ull;
}

// ------------------------------------------------------------------ Q/K/V of the block rows
// part: [splits][R][qw + 2 kvw] -> q (rotated), k_blk (rotated), v_blk
template <typename T>
__global__ void k_qkv_finish(const float* __restrict__ part, int splits, int R, int n_q, int n_kv, int hd,
                             const float* __restrict__ rope_blk, T* __restrict__ q, T* __restrict__ kb,
                             T* __restrict__ vb, int hpb, const T* __restrict__ g_q, const T* __restrict__ g_k,
                             float eps) {
  cod_pdl_prologue();
  // A block covers hpb heads of one row; hd / 8 threads per head, each owning 4 consecutive
  // elements of the lower half and their partners in the upper half (the pairs RoPE mixes).
  // Heads 0..n_q-1 are q, then n_kv heads of k (both rotated), then n_kv heads of v.
  // With per-head norms (g_q, g_k non-null) a head's threads first share its sum of squares.
  const int half = hd >> 1, tph = half >> 2;
  const int r = blockIdx.x, hh = blockIdx.y * hpb + threadIdx.x / tph, j = (threadIdx.x % tph) * 4;
  const bool live = hh < n_q + 2 * n_kv;            // whole warps stay for the shuffles
  const int qw = n_q * hd, kvw = n_kv * hd, ldc = qw + 2 * kvw;
  const float* p = part + static_cast<size_t>(r) * ldc + (live ? hh : 0) * hd + j;
  const size_t slab = static_cast<size_t>(R) * ldc;
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
  if (live) {
    // every slab's two loads are requested before the first sum (same order of sums)
#pragma unroll
    for (int s = 0; s < COD_MAX_SPLITS; ++s)
      if (s < splits) {
        a = f4_add(a, *reinterpret_cast<const float4*>(p + s * slab));
        b = f4_add(b, *reinterpret_cast<const float4*>(p + s * slab + half));
      }
    for (int s = COD_MAX_SPLITS; s < splits; ++s) {
      a = f4_add(a, *reinterpret_cast<const float4*>(p + s * slab));
      b = f4_add(b, *reinterpret_cast<const float4*>(p + s * slab + half));
    }
  }
  // The partial sums are dead once summed: the lines are dropped from L2 instead of being written back to HBM
  // later, under some HBM-bound kernel. Eight consecutive lanes share a 128-byte line; the first of them drops it
  // after the warp has met (all of the line's reads are then complete).
  if ((half & 31) == 0 && gridDim.x > COD_DROP_MIN_ROWS) {
    __syncwarp();
    const int g8 = threadIdx.x & 7;                  // the eight lanes share the drops: line (s, half) to lane 2 s + half
    if (live)
      for (int idx = g8; idx < 2 * splits; idx += 8) cod_discard_line(p - 4 * g8 + (idx >> 1) * slab + (idx & 1) * half);
  }
  const bool rot = hh < n_q + n_kv;
  const T* gain = hh < n_q ? g_q : (rot ? g_k : nullptr);
  if (g_q != nullptr) {                               // block-uniform: every lane takes the shuffles
    const float ss = group_sum(f4_ss(a) + f4_ss(b), tph);
    if (live && gain != nullptr) {
      const float sc = rsqrtf(ss / static_cast<float>(hd) + eps);
      a = f4_scale_gain(a, sc, cod_ld4(gain + j));
      b = f4_scale_gain(b, sc, cod_ld4(gain + half + j));
    }
  }
  if (!live) return;
  T* dst = hh < n_q ? q + static_cast<size_t>(r) * qw + hh * hd
                    : (rot ? kb + static_cast<size_t>(r) * kvw + (hh - n_q) * hd
                           : vb + static_cast<size_t>(r) * kvw + (hh - n_q - n_kv) * hd);
  if (rot) {
    const float* cs = rope_blk + static_cast<size_t>(r) * hd;
    const float4 c = *reinterpret_cast<const float4*>(cs + j), sn = *reinterpret_cast<const float4*>(cs + half + j);
    cod_st4(dst + j, make_float4(a.x * c.x - b.x * sn.x, a.y * c.y - b.y * sn.y, a.z * c.z - b.z * sn.z, a.w * c.w - b.w * sn.w));
    cod_st4(dst + j + half, make_float4(b.x * c.x + a.x * sn.x, b.y * c.y + a.y * sn.y, b.z * c.z + a.z * sn.z, b.w * c.w + a.w * sn.w));
  } else {
    cod_st4(dst + j, a);
    cod_st4(dst + j + half, b);
  }
}

// ------------------------------------------------------------------ gated MLP activation
// part: [splits][R][2 * d_ff] (gate columns, then up columns) -> h[r, j] = silu(gate) * up
template <typename T>
__global__ void k_swiglu_finish(const float* __restrict__ part, int splits, int R, int d_ff, T* __restrict__ h) {
  cod_pdl_prologue();
  const int r = blockIdx.x, j = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  if (j >= d_ff) return;
  const float* p = part + static_cast<size_t>(r) * 2 * d_ff + j;
  const size_t slab = static_cast<size_t>(R) * 2 * d_ff;
  float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
#pragma unroll 4
  for (int s = 0; s < splits; ++s) {
    g = f4_add(g, *reinterpret_cast<const float4*>(p + s * slab));
    u = f4_add(u, *reinterpret_cast<const float4*>(p + s * slab + d_ff));
  }
  cod_st4(h + static_cast<size_t>(r) * d_ff + j,
          make_float4(g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y,
                      g.z / (1.f + expf(-g.z)) * u.z, g.w / (1.f + expf(-g.w)) * u.w));
}

// Rotates caller-supplied q / k_blk (the stand-alone attention entry point).
template <typename T>
__global__ void k_rope_qk(const T* __restrict__ qin, const T* __restrict__ kin, int n_q, int n_kv, int hd,
                          const float* __restrict__ rope_blk, T* __restrict__ q, T* __restrict__ kb) {
  cod_pdl_prologue();
  const int r = blockIdx.x;
  const int qw = n_q * hd, kvw = n_kv * hd, half = hd >> 1;
  const float* cs = rope_blk + static_cast<size_t>(r) * hd;
  for (int e = threadIdx.x; e < (n_q + n_kv) * half; e += blockDim.x) {
    const int h = e / half, j = e - h * half;
    const T* src = h < n_q ? qin + static_cast<size_t>(r) * qw + h * hd : kin + static_cast<size_t>(r) * kvw + (h - n_q) * hd;
    T* dst = h < n_q ? q + static_cast<size_t>(r) * qw + h * hd : kb + static_cast<size_t>(r) * kvw + (h - n_q) * hd;
    const float a = cod_ld(src + j), b = cod_ld(src + j + half);
    const float c = cs[j], sn = cs[half + j];
    cod_st(dst + j, a * c - b * sn);
    cod_st(dst + j + half, b * c + a * sn);
  }
}

// ------------------------------------------------------------------ residual + norm
// x[r] += sum_splits part (if any); a[r] = N(x[r]) * gain
template <typename T, int NV>
__global__ void __launch_bounds__(1024) k_resid_norm(const float* __restrict__ part, int splits, int R, int D, float* x,
                             const T* __restrict__ gain, float eps, T* __restrict__ a, float* __restrict__ tap,
                             unsigned long long* __restrict__ amax) {
  cod_pdl_prologue();
  __shared__ float red[33];
  const int r = blockIdx.x;
  const int nv = D >> 2;
  float4 v[NV];
  float ss = 0.f;
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    v[t] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < nv) v[t] = *reinterpret_cast<const float4*>(x + static_cast<size_t>(r) * D + 4 * j);
  }
  if (part) {
    if (NV == 1) {
      // one slot per thread: every slab's load is requested before the first sum (same order of sums)
#pragma unroll
      for (int s = 0; s < COD_MAX_SPLITS; ++s)
        if (s < splits && static_cast<int>(threadIdx.x) < nv)
          v[0] = f4_add(v[0], *reinterpret_cast<const float4*>(part + (static_cast<size_t>(s) * R + r) * D + 4 * threadIdx.x));
    }
#pragma unroll 4
    for (int s = NV == 1 ? COD_MAX_SPLITS : 0; s < splits; ++s) {   // slots inside, four slabs unrolled: their loads are in flight together
#pragma unroll
      for (int t = 0; t < NV; ++t) {
        const int j = threadIdx.x + t * blockDim.x;
        if (j < nv) v[t] = f4_add(v[t], *reinterpret_cast<const float4*>(part + (static_cast<size_t>(s) * R + r) * D + 4 * j));
      }
    }
  }
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    if (j < nv) {
      if (part) *reinterpret_cast<float4*>(x + static_cast<size_t>(r) * D + 4 * j) = v[t];   // without partials x is read-only
      if (tap) *reinterpret_cast<float4*>(tap + static_cast<size_t>(r) * D + 4 * j) = v[t];
      ss += f4_ss(v[t]);
    }
  }
  ss = cod_block_sum(ss, red);
  // the partial sums are dead: their lines leave L2 without a write-back (the block has met since their last read)
  if (part && (D & 31) == 0 && gridDim.x > COD_DROP_MIN_ROWS) {
#pragma unroll
    for (int t = 0; t < NV; ++t) {
      const int j = threadIdx.x + t * blockDim.x;
      if (j < nv)
        for (int s = j & 7; s < splits; s += 8) cod_discard_line(part + (static_cast<size_t>(s) * R + r) * D + 4 * (j & ~7));
    }
  }
  const float scale = rsqrtf(ss / static_cast<float>(D) + eps);
#pragma unroll
  for (int t = 0; t < NV; ++t) {
    const int j = threadIdx.x + t * blockDim.x;
    if (j < nv) {
      const float4 g = cod_ld4(gain + 4 * j);
      cod_st4(a + static_cast<size_t>(r) * D + 4 * j,
              make_float4(v[t].x * scale * g.x, v[t].y * scale * g.y, v[t].z * scale * g.z, v[t].w * scale * g.w));
    }
  }
  if (amax && threadIdx.x == 0) amax[r] = 0ull;
}

__global__ void k_finalize(const unsigned long long* __restrict__ amax, int R, int W, const int* __restrict__ bonus,
                           int* __restrict__ tok, int* __restrict__ next_draft, float* __restrict__ top_logit) {
  cod_pdl_prologue();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  const unsigned long long key = amax[r];
  const int t = cod_unpack_index(key);
  if (tok) tok[r] = t;
  if (top_logit) top_logit[r] = cod_unpack_logit(key);
  if (next_draft) next_draft[r] = (r % W == 0) ? bonus[r / W] : t;
}

}  // namespace

// One float4 slot per thread where the row allows it: these kernels are latency-bound, so the more
// independent loads a row has in flight the better.
static inline bool row_narrow(int D) { return D <= 4096; }
static inline int row_threads(int D) {
  if (!row_narrow(D)) return 1024;
  const int nt = ((D / 4 + 31) / 32) * 32;
  return nt < 128 ? 128 : nt;
}

#define DISPATCH_T(c, CALL_BF16, CALL_F32) \
  do {                                     \
    if ((c)->cfg.dtype == COD_BF16) { CALL_BF16; } else { CALL_F32; } \
  } while (0)

int cod_launch_gather_rows(cod_ctx* c, const void* src, const int* rows, const int* n_dev, int n_max, int width,
                           void* dst, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  if (n_max <= 0) return COD_OK;
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_gather_rows<__nv_bfloat16>, n_max, 256, 0, st, static_cast<const __nv_bfloat16*>(src), rows, n_dev, width, static_cast<__nv_bfloat16*>(dst))),
             (cod_launch_pdl(c, k_gather_rows<float>, n_max, 256, 0, st, static_cast<const float*>(src), rows, n_dev, width, static_cast<float*>(dst))));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_gather_grouped(cod_ctx* c, const void* src, const cod_split* sp, int S, int R, int width, void* dst, int* perm,
                              cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  if (R <= 0) return COD_OK;
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_gather_grouped<__nv_bfloat16>, R, 256, 0, st, static_cast<const __nv_bfloat16*>(src), sp->acc_rows, sp->acc_off + S, sp->rej_rows, width, static_cast<__nv_bfloat16*>(dst), perm)),
             (cod_launch_pdl(c, k_gather_grouped<float>, R, 256, 0, st, static_cast<const float*>(src), sp->acc_rows, sp->acc_off + S, sp->rej_rows, width, static_cast<float*>(dst), perm)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_fcE(cod_ctx* c, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_fcE<__nv_bfloat16>, c->D, 256, 0, st, static_cast<const __nv_bfloat16*>(c->w.fc), static_cast<const __nv_bfloat16*>(c->w.e_carry), c->D_in, c->fcE)),
             (cod_launch_pdl(c, k_fcE<float>, c->D, 256, 0, st, static_cast<const float*>(c->w.fc), static_cast<const float*>(c->w.e_carry), c->D_in, c->fcE)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_fc_finish(cod_ctx* c, const float* part, int splits, int n_rows, const int* n_rows_dev,
                         const int* a_rows, const int* carry_slot, float* tap_z, cudaStream_t st, int ldp, int dense_base,
                         int z_by_row) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  if (n_rows <= 0) return COD_OK;
  const int nt = row_threads(c->D);
  const int do_norm = (c->cfg.flags & COD_F_HIDDEN_NORM) ? 1 : 0;
  // F(E_carry) is added to rejected rows only in the embedding variant
  const float* fcE = (c->cfg.flags & (COD_F_NO_CARRY_EMBED | COD_F_REJ_PROJECTOR)) ? nullptr : c->fcE;
  if (ldp <= 0) ldp = c->D;
  if (row_narrow(c->D)) {
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_fc_finish<__nv_bfloat16, 1>, n_rows, nt, 0, st, part, splits, n_rows, n_rows_dev, a_rows, carry_slot, fcE, static_cast<const __nv_bfloat16*>(c->w.g_hidden), c->D, c->cfg.rms_eps, do_norm, static_cast<__nv_bfloat16*>(c->z), (a_rows && !z_by_row) ? 1 : 0, tap_z, ldp, dense_base)),
               (cod_launch_pdl(c, k_fc_finish<float, 1>, n_rows, nt, 0, st, part, splits, n_rows, n_rows_dev, a_rows, carry_slot, fcE, static_cast<const float*>(c->w.g_hidden), c->D, c->cfg.rms_eps, do_norm, static_cast<float*>(c->z), (a_rows && !z_by_row) ? 1 : 0, tap_z, ldp, dense_base)));
  } else {
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_fc_finish<__nv_bfloat16, ROW_WIDE_NV>, n_rows, nt, 0, st, part, splits, n_rows, n_rows_dev, a_rows, carry_slot, fcE, static_cast<const __nv_bfloat16*>(c->w.g_hidden), c->D, c->cfg.rms_eps, do_norm, static_cast<__nv_bfloat16*>(c->z), (a_rows && !z_by_row) ? 1 : 0, tap_z, ldp, dense_base)),
               (cod_launch_pdl(c, k_fc_finish<float, ROW_WIDE_NV>, n_rows, nt, 0, st, part, splits, n_rows, n_rows_dev, a_rows, carry_slot, fcE, static_cast<const float*>(c->w.g_hidden), c->D, c->cfg.rms_eps, do_norm, static_cast<float*>(c->z), (a_rows && !z_by_row) ? 1 : 0, tap_z, ldp, dense_base)));
  }
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_kv_finish(cod_ctx* c, const float* part, int splits, int n_rows, const int* n_rows_dev,
                         const int* a_rows, const cod_split* sp, void* J, const cod_state* ds, int R_total,
                         cudaStream_t st, int dense_base) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  if (n_rows <= 0) return COD_OK;
  const cod_config& f = c->cfg;
  dim3 grid(n_rows, f.n_layers);
  const int to_state = ds ? 1 : 0;
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_kv_finish<__nv_bfloat16>, grid, 128, 0, st, part, splits, n_rows, n_rows_dev, a_rows, c->rope_win, f.n_layers, f.n_kv_heads, f.head_dim, static_cast<__nv_bfloat16*>(J), R_total, sp->commit_slot, sp->carry_slot, ds ? static_cast<__nv_bfloat16*>(ds->kv_pool) : nullptr, ds ? static_cast<__nv_bfloat16*>(ds->carry_kv) : nullptr, f.page_size, f.n_pages, f.block, f.max_batch, to_state, (f.flags & COD_F_QK_NORM) ? static_cast<const __nv_bfloat16*>(c->w.g_knorm) : nullptr, f.rms_eps, c->carry_cap, c->carry_base, dense_base)),
             (cod_launch_pdl(c, k_kv_finish<float>, grid, 128, 0, st, part, splits, n_rows, n_rows_dev, a_rows, c->rope_win, f.n_layers, f.n_kv_heads, f.head_dim, static_cast<float*>(J), R_total, sp->commit_slot, sp->carry_slot, ds ? static_cast<float*>(ds->kv_pool) : nullptr, ds ? static_cast<float*>(ds->carry_kv) : nullptr, f.page_size, f.n_pages, f.block, f.max_batch, to_state, (f.flags & COD_F_QK_NORM) ? static_cast<const float*>(c->w.g_knorm) : nullptr, f.rms_eps, c->carry_cap, c->carry_base, dense_base)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_scatter(cod_ctx* c, const void* J, const cod_split* sp, int S, int mode, const cod_state* ds,
                       cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const cod_config& f = c->cfg;
  const int R = S * f.block;
  dim3 grid(R, f.n_layers);
  const int use_carry = mode == COD_CARRY;
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_scatter_kv<__nv_bfloat16>, grid, 128, 0, st, static_cast<const __nv_bfloat16*>(J), R, f.n_kv_heads, f.head_dim, sp->commit_slot, sp->carry_slot, static_cast<__nv_bfloat16*>(ds->kv_pool), static_cast<__nv_bfloat16*>(ds->carry_kv), f.page_size, f.n_pages, f.block, f.max_batch, use_carry, c->carry_cap, c->carry_base)),
             (cod_launch_pdl(c, k_scatter_kv<float>, grid, 128, 0, st, static_cast<const float*>(J), R, f.n_kv_heads, f.head_dim, sp->commit_slot, sp->carry_slot, static_cast<float*>(ds->kv_pool), static_cast<float*>(ds->carry_kv), f.page_size, f.n_pages, f.block, f.max_batch, use_carry, c->carry_cap, c->carry_base)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_update_lens(cod_ctx* c, const cod_split* sp, int S, int mode, const cod_state* ds, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const LensUpdate u{sp->accept_len, S, c->cfg.block, mode, c->cfg.max_pages_per_seq * c->cfg.page_size,
                     ds->committed_len, ds->carry_len, c->status, c->carry_base};
  cod_launch_pdl(c, k_update_lens, (S + 127) / 128, 128, 0, st, u);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_carry_age(cod_ctx* c, const cod_split* sp, int S, int mode, const cod_state* ds, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const cod_config& f = c->cfg;
  const int k = c->carry_cap / f.block;
  cod_launch_pdl(c, k_carry_age_hist, (S + 127) / 128, 128, 0, st, sp->accept_len, ds->carry_len, S, f.block, k, mode,
                 ds->carry_hist, c->carry_base, c->carry_drop);
  COD_CHECK_LAUNCH(c);
  const dim3 grid(S, f.n_kv_heads * 2, f.n_layers);
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_carry_shift<__nv_bfloat16>, grid, 128, 0, st, static_cast<__nv_bfloat16*>(ds->carry_kv), c->carry_base, c->carry_drop, f.max_batch, f.n_kv_heads, c->carry_cap, f.head_dim)),
             (cod_launch_pdl(c, k_carry_shift<float>, grid, 128, 0, st, static_cast<float*>(ds->carry_kv), c->carry_base, c->carry_drop, f.max_batch, f.n_kv_heads, c->carry_cap, f.head_dim)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_embed_norm(cod_ctx* c, const int32_t* bonus, int S, cudaStream_t st, const cod_split* sp, int mode,
                          const cod_state* ds) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const cod_config& f = c->cfg;
  const int R = S * f.block;
  LensUpdate u{};                                   // sp == null: no length update rides along
  if (sp) u = LensUpdate{sp->accept_len, S, f.block, mode, f.max_pages_per_seq * f.page_size, ds->committed_len,
                         ds->carry_len, c->status, c->carry_base};
  if (row_narrow(c->D)) {
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_embed_norm<__nv_bfloat16, 1>, R, row_threads(c->D), 0, st, static_cast<const __nv_bfloat16*>(c->w.emb), bonus, f.block, f.mask_token_id, f.vocab, static_cast<const __nv_bfloat16*>(c->w.g_attn), c->D, f.rms_eps, c->x, static_cast<__nv_bfloat16*>(c->a), c->amax, u)),
               (cod_launch_pdl(c, k_embed_norm<float, 1>, R, row_threads(c->D), 0, st, static_cast<const float*>(c->w.emb), bonus, f.block, f.mask_token_id, f.vocab, static_cast<const float*>(c->w.g_attn), c->D, f.rms_eps, c->x, static_cast<float*>(c->a), c->amax, u)));
  } else {
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_embed_norm<__nv_bfloat16, ROW_WIDE_NV>, R, row_threads(c->D), 0, st, static_cast<const __nv_bfloat16*>(c->w.emb), bonus, f.block, f.mask_token_id, f.vocab, static_cast<const __nv_bfloat16*>(c->w.g_attn), c->D, f.rms_eps, c->x, static_cast<__nv_bfloat16*>(c->a), c->amax, u)),
               (cod_launch_pdl(c, k_embed_norm<float, ROW_WIDE_NV>, R, row_threads(c->D), 0, st, static_cast<const float*>(c->w.emb), bonus, f.block, f.mask_token_id, f.vocab, static_cast<const float*>(c->w.g_attn), c->D, f.rms_eps, c->x, static_cast<float*>(c->a), c->amax, u)));
  }
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_qkv_finish(cod_ctx* c, const float* part, int splits, int R, int layer, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const cod_config& f = c->cfg;
  // heads per block: as many (up to 8) as still leave a couple of blocks per SM; whole warps always
  const int nh = f.n_q_heads + 2 * f.n_kv_heads, tph = f.head_dim / 8;
  const int hpb_min = 32 / tph > 1 ? 32 / tph : 1;
  int hpb = 8;
  while (hpb > hpb_min && R * ((nh + hpb - 1) / hpb) < 2 * c->n_sm) hpb >>= 1;
  const dim3 grid(R, (nh + hpb - 1) / hpb);
  const bool qk = (f.flags & COD_F_QK_NORM) != 0;
  const size_t goff = static_cast<size_t>(layer) * f.head_dim;
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_qkv_finish<__nv_bfloat16>, grid, tph * hpb, 0, st, part, splits, R, f.n_q_heads, f.n_kv_heads, f.head_dim, c->rope_blk, static_cast<__nv_bfloat16*>(c->q), static_cast<__nv_bfloat16*>(c->kb), static_cast<__nv_bfloat16*>(c->vb), hpb, qk ? static_cast<const __nv_bfloat16*>(c->w.g_qnorm) + goff : nullptr, qk ? static_cast<const __nv_bfloat16*>(c->w.g_knorm) + goff : nullptr, f.rms_eps)),
             (cod_launch_pdl(c, k_qkv_finish<float>, grid, tph * hpb, 0, st, part, splits, R, f.n_q_heads, f.n_kv_heads, f.head_dim, c->rope_blk, static_cast<float*>(c->q), static_cast<float*>(c->kb), static_cast<float*>(c->vb), hpb, qk ? static_cast<const float*>(c->w.g_qnorm) + goff : nullptr, qk ? static_cast<const float*>(c->w.g_knorm) + goff : nullptr, f.rms_eps)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

// ------------------------------------------------------------------ reference logits of the rank head
// ref[r] = a[r] . Emb[tok[r]] in float (the operands the contraction reads); out-of-range tokens are
// flagged and replaced by 0; the row's count starts at zero.
template <typename T>
__global__ void k_rank_ref(const T* __restrict__ a, const T* __restrict__ emb, const int32_t* __restrict__ ref_tok,
                           int D, int vocab, float* __restrict__ ref, int32_t* __restrict__ tok_clean,
                           int32_t* __restrict__ rank, uint32_t* status) {
  cod_pdl_prologue();
  __shared__ float red[33];
  const int r = blockIdx.x;
  int tok = ref_tok[r];
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) atomicOr(status, COD_DEV_BAD_TOKEN);
    tok = 0;
  }
  const T* x = a + static_cast<size_t>(r) * D;
  const T* e = emb + static_cast<size_t>(tok) * D;
  float acc = 0.f;
  for (int j = threadIdx.x * 4; j < D; j += blockDim.x * 4) {       // D % 8 == 0
    const float4 u = cod_ld4(x + j), v = cod_ld4(e + j);
    acc = fmaf(u.x, v.x, fmaf(u.y, v.y, fmaf(u.z, v.z, fmaf(u.w, v.w, acc))));
  }
  acc = cod_block_sum(acc, red);
  if (threadIdx.x == 0) { ref[r] = acc; tok_clean[r] = tok; rank[r] = 0; }
}

int cod_launch_rank_ref(cod_ctx* c, int n_rows, const int32_t* ref_tok, float* ref, int32_t* tok_clean,
                        int32_t* rank, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_rank_ref<__nv_bfloat16>, n_rows, 256, 0, st, static_cast<const __nv_bfloat16*>(c->a), static_cast<const __nv_bfloat16*>(c->w.emb), ref_tok, c->D, c->cfg.vocab, ref, tok_clean, rank, c->status)),
             (cod_launch_pdl(c, k_rank_ref<float>, n_rows, 256, 0, st, static_cast<const float*>(c->a), static_cast<const float*>(c->w.emb), ref_tok, c->D, c->cfg.vocab, ref, tok_clean, rank, c->status)));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_swiglu_finish(cod_ctx* c, const float* part, int splits, int R, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const int d_ff = c->cfg.d_ff;
  const dim3 grid(R, (d_ff / 4 + 255) / 256);
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_swiglu_finish<__nv_bfloat16>, grid, 256, 0, st, part, splits, R, d_ff, static_cast<__nv_bfloat16*>(c->hmid))),
             (cod_launch_pdl(c, k_swiglu_finish<float>, grid, 256, 0, st, part, splits, R, d_ff, static_cast<float*>(c->hmid))));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

// rope_blk must already hold the block rows' tables
int cod_launch_rope_qk(cod_ctx* c, const void* q, const void* k, const int32_t* committed_len, int S, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  (void)committed_len;
  const cod_config& f = c->cfg;
  const int R = S * f.block;
  DISPATCH_T(c,
             (cod_launch_pdl(c, k_rope_qk<__nv_bfloat16>, R, 256, 0, st, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), f.n_q_heads, f.n_kv_heads, f.head_dim, c->rope_blk, static_cast<__nv_bfloat16*>(c->q), static_cast<__nv_bfloat16*>(c->kb))),
             (cod_launch_pdl(c, k_rope_qk<float>, R, 256, 0, st, static_cast<const float*>(q), static_cast<const float*>(k), f.n_q_heads, f.n_kv_heads, f.head_dim, c->rope_blk, static_cast<float*>(c->q), static_cast<float*>(c->kb))));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_resid_norm(cod_ctx* c, const float* part, int splits, int R, float* x, const void* gain,
                          float* tap_x, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  // More rows than one wave of one-slot-per-thread blocks holds (three 640-thread blocks per SM at D = 2560):
  // two slots per thread and half the threads, so every row is resident at once.
  const int nt1 = row_threads(c->D);
  if (row_narrow(c->D) && R > (2048 / nt1) * c->n_sm && nt1 >= 256) {
    const int nt2 = ((c->D / 8 + 31) / 32) * 32;
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_resid_norm<__nv_bfloat16, 2>, R, nt2, 0, st, part, splits, R, c->D, x, static_cast<const __nv_bfloat16*>(gain), c->cfg.rms_eps, static_cast<__nv_bfloat16*>(c->a), tap_x, c->amax)),
               (cod_launch_pdl(c, k_resid_norm<float, 2>, R, nt2, 0, st, part, splits, R, c->D, x, static_cast<const float*>(gain), c->cfg.rms_eps, static_cast<float*>(c->a), tap_x, c->amax)));
  } else if (row_narrow(c->D)) {
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_resid_norm<__nv_bfloat16, 1>, R, row_threads(c->D), 0, st, part, splits, R, c->D, x, static_cast<const __nv_bfloat16*>(gain), c->cfg.rms_eps, static_cast<__nv_bfloat16*>(c->a), tap_x, c->amax)),
               (cod_launch_pdl(c, k_resid_norm<float, 1>, R, row_threads(c->D), 0, st, part, splits, R, c->D, x, static_cast<const float*>(gain), c->cfg.rms_eps, static_cast<float*>(c->a), tap_x, c->amax)));
  } else {
    DISPATCH_T(c,
               (cod_launch_pdl(c, k_resid_norm<__nv_bfloat16, ROW_WIDE_NV>, R, row_threads(c->D), 0, st, part, splits, R, c->D, x, static_cast<const __nv_bfloat16*>(gain), c->cfg.rms_eps, static_cast<__nv_bfloat16*>(c->a), tap_x, c->amax)),
               (cod_launch_pdl(c, k_resid_norm<float, ROW_WIDE_NV>, R, row_threads(c->D), 0, st, part, splits, R, c->D, x, static_cast<const float*>(gain), c->cfg.rms_eps, static_cast<float*>(c->a), tap_x, c->amax)));
  }
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

int cod_launch_finalize(cod_ctx* c, int R, int W, const int32_t* bonus, int32_t* tok, int32_t* next_draft,
                        float* top_logit, cudaStream_t st) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  cod_launch_pdl(c, k_finalize, (R + 127) / 128, 128, 0, st, c->amax, R, W, bonus, tok, next_draft, top_logit);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}
