// Weight-streaming GEMM for many token rows (more than 128): the same swap-AB scheme as
// k_gemm_tc, but two CTAs of a thread-block cluster (two SMs) work on one 256 x 256 tile with
// tcgen05.mma.cta_group::2:
//   C[i, n] = sum_k A[i, k] * B[n, k]     A: activations [rows, K], B: weights [N, K].
// Each CTA stages its own 128 weight rows and its own half (128) of the 256 token rows, so per
// unit of tensor work every SM pulls half as many operand bytes through its TMA engine as a
// single-CTA 128 x 256 tile does - the engine (about 36 B/clk per SM), not the tensor pipe,
// is what limits the single-CTA kernel once the GEMM is compute-bound.
//
// Protocol (rank 0 of the pair is the leader):
//   * both CTAs: TMA producer warp loads its tiles with the cta_group::2 form of the copy, which
//     signals the LEADER's "full" barrier; the leader expects the bytes of both CTAs;
//   * leader only: one thread issues the MMAs (M = 256 spans both CTAs' tensor memory) and commits
//     with a cluster-wide arrive to the "empty" barrier of both CTAs (and, at the end, to both
//     "accumulator ready" barriers);
//   * both CTAs: all eight warps read the CTA's own 128 accumulator rows back (two warps per 32 lanes,
//     each taking half of the token columns).
// No load is delivered to more than one CTA. Waits are bounded as in k_gemm_tc; the only
// unbounded synchronisation is the hardware cluster barrier, which every thread reaches
// unconditionally.
#include "tc_common.cuh"

namespace {
// A weight tile is read once per launch: fetched with an L2 evict-first hint it leaves the cache before the token
// operand every pair re-reads and before the float partial sums the finishing kernel is about to read.
__device__ __forceinline__ void tma_load_2d_pair_stream(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t leader_bar) {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(leader_bar), "l"(pol) : "memory");
}

using namespace tc;

constexpr int BM = 128;       // weight rows per CTA (256 per pair)
constexpr int BK = 64;
constexpr int UK = 16;
constexpr int NT = 256;       // token rows per pair = MMA N; each CTA stages NT / 2 of them
constexpr int NTHREADS = 256;   // 8 warps: all of them read the accumulator back; warps 4 and 5 first produce / issue
constexpr uint32_t A_TILE_BYTES = BM * BK * 2;          // 16 KB
constexpr uint32_t B_TILE_BYTES = (NT / 2) * BK * 2;    // 16 KB
constexpr int MAX_STAGES = 6;   // one accumulator: 6 stages of 32 KB; two: 4 stages of 48 KB

struct Tc2Params {
  int K, kb_total, kb_per_split;
  int n_rows;
  const int* n_rows_dev;
  const int* group_split_dev; // two segments grouped by row: segment 0 owns rows [0, *g), segment 1 rows [*g, n_rows); same columns
  int pair_end[3];            // cumulative count of 256-row tile pairs after each weight segment
  int seg_N[3];
  int n_seg;
  int n_tiles_n;              // token tiles
  int tail_pairs;             // the last tail_pairs weight tiles run as two launches of one accumulator each (see the launcher)
  int n_acc;                  // accumulators per pair: 1 (256 token rows) or 2 (512)
  int stages;
  int staged;                 // epilogue transposes through shared memory (needs 16-byte aligned feature runs)
  float* C;
  int ldc;
  unsigned long long* amax;
  float2* lse_part;           // sampling form of the argmax epilogue (null: plain argmax)
  uint32_t sample_state;
  uint32_t* status;
};


// SAMPLE selects the sampling form of the argmax epilogue at compile time (see k_gemm_tc).
template <bool SAMPLE>
__global__ void __launch_bounds__(NTHREADS, 1)
k_gemm_tc2(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
           const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_a, const Tc2Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t STAGE_BYTES = A_TILE_BYTES + p.n_acc * B_TILE_BYTES;
  const int STAGES = p.stages;
  const int NTOK = p.n_acc * NT;                                       // token rows of this pair's tile
  const uint32_t TMEM_COLS = static_cast<uint32_t>(NTOK);
  uint8_t* ctl = sm + STAGES * STAGE_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ctl);               // [STAGES], used in the leader
  uint64_t* empty_bar = full_bar + 8;                                  // [STAGES]
  uint64_t* acc_bar = full_bar + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(full_bar + 17);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned long long* red = reinterpret_cast<unsigned long long*>(full_bar + 18);   // [4][NT]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = blockIdx.x;                    // position in the pair; 0 leads
  const int n_tile = blockIdx.y % p.n_tiles_n, split = blockIdx.z;
  int pair = blockIdx.y / p.n_tiles_n;
  int half = -1;                                  // >= 0: this pair works on one accumulator (256 token rows) of a tail tile
  if (p.tail_pairs > 0) {
    const int whole = p.pair_end[p.n_seg - 1] - p.tail_pairs;
    if (pair >= whole) { half = (pair - whole) & 1; pair = whole + ((pair - whole) >> 1); }
  }
  const int i0 = n_tile * NTOK;

  int sidx = 0;
  while (sidx < p.n_seg - 1 && pair >= p.pair_end[sidx]) ++sidx;
  const int pair_in_seg = pair - (sidx ? p.pair_end[sidx - 1] : 0);
  const int f0 = pair_in_seg * 2 * BM + rank * BM;           // this CTA's first weight row within the segment
  int col0 = f0;
  for (int s = 0; s < sidx; ++s) col0 += p.seg_N[s];
  const int seg_N = p.seg_N[sidx];
  const CUtensorMap* map_w = sidx == 0 ? &map_w0 : (sidx == 1 ? &map_w1 : &map_w2);
  const int kb0 = split * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
  const int n_pre = min(STAGES, kb1 - kb0);       // stages whose weight tile is requested ahead of the dependency

  // ---- before the dependency on the previous kernel resolves: set up, and start streaming the
  // weights (nothing in the stream writes them). Their bytes are counted on the leader's stage
  // barrier before its expect_tx below, which the transaction count allows.
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(full_bar + s), 1); mbar_init(smem_u32(empty_bar + s), 1); }
    mbar_init(smem_u32(acc_bar), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int t = threadIdx.x; t < 4 * NTOK; t += NTHREADS) red[t] = 0ull;
  if (warp == 5) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // the partner's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp == 4 && lane == 0)
    for (int it = 0; it < n_pre; ++it)
      tma_load_2d_pair_stream(base + it * STAGE_BYTES, map_w, (kb0 + it) * BK, f0, smem_u32(full_bar + it) & PEER_MASK);

  cod_pdl_prologue();
  const int n_rows = p.n_rows_dev ? min(*p.n_rows_dev, p.n_rows) : p.n_rows;
  int row_lo = 0, row_hi = n_rows;                // token rows this tile's weight segment is meant for
  if (p.group_split_dev != nullptr) {
    const int g = max(0, min(*p.group_split_dev, n_rows));
    if (sidx == 0) row_hi = g; else row_lo = g;
    col0 = f0;                                    // both groups' results share the columns
  }
  if (half >= 0) { row_lo = max(row_lo, half * NT); row_hi = min(row_hi, (half + 1) * NT); }
  // NOTE: both CTAs of a pair take the same decision here (it depends on the pair's tile only)
  const int n_kb = (i0 < row_hi && i0 + NTOK > row_lo) ? kb1 - kb0 : 0;   // 0: no token rows here, only the requested weights to absorb
  // accumulators whose 256 token rows miss this segment's row range altogether are neither fed nor multiplied
  // (a contraction grouped by row: the group boundary usually leaves one of the two accumulators empty)
  uint32_t acc_on = 0;
  for (int a = 0; a < p.n_acc; ++a)
    if (i0 + a * NT < row_hi && i0 + (a + 1) * NT > row_lo) acc_on |= 1u << a;
  const uint32_t stage_tx = 2 * (A_TILE_BYTES + static_cast<uint32_t>(__popc(acc_on)) * B_TILE_BYTES);

  if (warp == 4) {
    if (lane == 0) {
      if (n_kb == 0 && rank == 0) {
        for (int it = 0; it < n_pre; ++it) {
          mbar_expect_tx(smem_u32(full_bar + it), 2 * A_TILE_BYTES);
          if (!mbar_wait(smem_u32(full_bar + it), 0, abort_flag, p.status)) break;
        }
      }
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % STAGES, use = it / STAGES;
        if (use > 0 && !mbar_wait(smem_u32(empty_bar + s), (use - 1) & 1, abort_flag, p.status)) break;
        const uint32_t fb = smem_u32(full_bar + s);
        if (rank == 0) mbar_expect_tx(fb, stage_tx);            // both CTAs' bytes land on the leader's barrier
        const uint32_t a_dst = base + s * STAGE_BYTES;
        const int k = (kb0 + it) * BK;
        if (it >= n_pre) tma_load_2d_pair_stream(a_dst, map_w, k, f0, fb & PEER_MASK);
        for (int a = 0; a < p.n_acc; ++a)      // accumulator a covers tokens [i0 + a*256, +256): this CTA stages its half
          if (acc_on & (1u << a)) tma_load_2d_pair(a_dst + A_TILE_BYTES + a * B_TILE_BYTES, &map_a, k, i0 + a * NT + rank * (NT / 2), fb & PEER_MASK);
      }
    }
  } else if (warp == 5) {
    if (lane == 0 && rank == 0) {
      // bf16 x bf16 -> float, K-major operands, M = 256 (both CTAs), N = 256
      const uint32_t idesc = instr_desc(2 * BM, NT, 0);
      bool ok = true;
      for (int it = 0; it < n_kb && ok; ++it) {
        const int s = it % STAGES, use = it / STAGES;
        ok = mbar_wait(smem_u32(full_bar + s), use & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = base + s * STAGE_BYTES;
        const uint64_t a_desc = desc_kmajor_sw128(a_addr);
        for (int a = 0; a < p.n_acc; ++a) {
          if (!(acc_on & (1u << a))) continue;
          const uint64_t b_desc = desc_kmajor_sw128(a_addr + A_TILE_BYTES + a * B_TILE_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UK; ++k)
            umma_bf16_pair(tmem_base + a * NT, a_desc + (k * UK * 2 >> 4), b_desc + (k * UK * 2 >> 4), idesc, (it | k) ? 1u : 0u);
        }
        umma_commit_pair(smem_u32(empty_bar + s), 3);
      }
      if (ok && n_kb > 0) umma_commit_pair(smem_u32(acc_bar), 3);
    }
  }
  __syncwarp();

  // ---------------------------------------------------- epilogue, all 8 warps
  // Warp w reads tensor-memory lanes 32 * (w % 4) .. +31 (the only lanes it may touch); warps 0-3
  // take the first half of the token columns, warps 4-7 the second.
  if (n_kb > 0) {
    // one decision for everyone (the warps meet at named barriers below)
    const bool ok = __syncthreads_and(mbar_wait(smem_u32(acc_bar), 0, abort_flag, p.status)) != 0;
    tc_fence_after();
    const int qw = warp & 3, grp = warp >> 2;
    const int c_begin = grp * (NTOK / 2), c_end = c_begin + NTOK / 2;
    const int f = f0 + qw * 32 + lane;
    const bool f_ok = f < seg_N;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(qw * 32) << 16);
    if (ok && p.amax == nullptr && p.staged) {
      // The accumulator has features on lanes and tokens on columns; C wants a token's features
      // contiguous. Each group of four warps transposes 32 tokens at a time through the (now idle)
      // pipeline buffers and stores whole 512-byte feature runs: two 16 KB buffers per group, one
      // named barrier of the group per chunk.
      float* C = p.C + static_cast<size_t>(split) * p.n_rows * p.ldc + col0;
      float* stage = reinterpret_cast<float*>(sm) + grp * (2 * 32 * BM);
      const int f_left = seg_N - f0;                       // features of this CTA that exist
      for (int c = c_begin, q = 0; c < c_end && i0 + c < row_hi; c += 32, q ^= 1) {
        if (i0 + c + 32 <= row_lo) continue;               // (the whole group of four warps skips together)
        uint32_t v[32];
        tmem_ld32(t_lane + c, v);
        float* buf = stage + q * (32 * BM);
#pragma unroll
        for (int j = 0; j < 32; ++j) buf[j * BM + qw * 32 + lane] = __uint_as_float(v[j]);
        asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory");
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const int tok = qw * 8 + t, i = i0 + c + tok;
          if (i >= row_lo && i < row_hi && lane * 4 < f_left)
            *reinterpret_cast<float4*>(C + static_cast<size_t>(i) * p.ldc + lane * 4) =
                *reinterpret_cast<const float4*>(buf + tok * BM + lane * 4);
        }
      }
    } else if (ok && p.amax == nullptr) {
      float* C = p.C + static_cast<size_t>(split) * p.n_rows * p.ldc;
      for (int c = c_begin; c < c_end; c += 16) {
        if (i0 + c >= row_hi) break;
        if (i0 + c + 16 <= row_lo) continue;
        uint32_t v[16];
        tmem_ld16(t_lane + c, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int i = i0 + c + j;
          if (f_ok && i >= row_lo && i < row_hi) C[static_cast<size_t>(i) * p.ldc + col0 + qw * 32 + lane] = __uint_as_float(v[j]);
        }
      }
    } else if (SAMPLE && ok) {
      // sampling form: Gumbel noise on every logit before the argmax, and soft-max partials per column.
      // Scratch in the idle pipeline buffers: row states, then per-warp (m, sum) of every column.
      uint32_t* hrow = reinterpret_cast<uint32_t*>(sm);
      float* red_m = reinterpret_cast<float*>(sm + 4096);
      float* red_s = red_m + 4 * NTOK;
      for (int t = c_begin + qw * 32 + lane; t < c_end; t += 128) hrow[t] = mix32(p.sample_state + static_cast<uint32_t>(i0 + t));
      asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory");
      for (int c = c_begin; c < c_end; c += 32) {
        if (i0 + c >= row_hi) break;
        if (i0 + c + 32 <= row_lo) continue;
        uint32_t v[32];
        tmem_ld32(t_lane + c, v);
        unsigned long long best;
        float m_ref, s_sum;
        sample_chunk(v, f_ok, static_cast<uint32_t>(col0 + qw * 32 + lane), hrow + c, lane, best, m_ref, s_sum);
        red[qw * NTOK + c + lane] = best;
        red_m[qw * NTOK + c + lane] = m_ref;
        red_s[qw * NTOK + c + lane] = s_sum;
      }
    } else if (ok) {
      const unsigned long long low = static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<unsigned>(col0 + qw * 32 + lane));
      for (int c = c_begin; c < c_end; c += 32) {
        if (i0 + c >= row_hi) break;
        if (i0 + c + 32 <= row_lo) continue;
        uint32_t v[32];
        tmem_ld32(t_lane + c, v);
        unsigned long long k[32];
#pragma unroll
        for (int j = 0; j < 32; ++j)
          k[j] = f_ok ? ((static_cast<unsigned long long>(order_key(__uint_as_float(v[j]))) << 32) | low) : 0ull;
        red[qw * NTOK + c + lane] = warp_colmax32(k, lane);
      }
    }
  }

  // ---------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  } else if (p.amax != nullptr && n_kb > 0) {
    for (int t = threadIdx.x; t < NTOK; t += NTHREADS) {
      if (i0 + t >= row_lo && i0 + t < row_hi) {
        unsigned long long best = red[t];
#pragma unroll
        for (int w = 1; w < 4; ++w) best = red[w * NTOK + t] > best ? red[w * NTOK + t] : best;
        if (best) atomicMax(p.amax + i0 + t, best);
        if (SAMPLE) {                                  // this tile's soft-max partial of token row i0 + t
          const float* red_m = reinterpret_cast<const float*>(sm + 4096);
          const float* red_s = red_m + 4 * NTOK;
          float m = red_m[t];
#pragma unroll
          for (int w = 1; w < 4; ++w) m = fmaxf(m, red_m[w * NTOK + t]);
          float sum = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w)
            if (red_m[w * NTOK + t] > -INFINITY) sum += red_s[w * NTOK + t] * __expf(red_m[w * NTOK + t] - m);
          p.lse_part[static_cast<size_t>(col0 / BM) * p.n_rows + i0 + t] = make_float2(m, sum);
        }
      }
    }
  }
  cluster_sync_all();                 // neither CTA frees tensor memory or exits while the other may still touch it
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}


}  // namespace

// Modelled time of one launch in SM cycles, from device-side cycle stamps of this kernel:
//   per CTA pair: ~7500 cycles before the first MMA (setup, first operands), then per 64-wide
//   k-block ~760 cycles with one accumulator (the operand fetch of 32 KB per SM is the limit) and
//   ~1000 with two (48 KB per SM, the tensor pipe is the limit), then ~3000 cycles of epilogue per
//   accumulator; pairs run in waves of n_sm / 2;
//   every split beyond the first costs one more float slab written here and read by the
//   finishing kernel (~30 bytes per cycle per SM through L2).
void cod_plan_gemm_tc2(int n_sm, int n_out, int K, int rows, int max_splits, int fixed_splits, int* splits_out,
                       int* n_acc_out) {
  const int kb = (K + BK - 1) / BK;
  const int pairs = (n_out + 2 * BM - 1) / (2 * BM);
  const int per_wave = n_sm / 2 > 0 ? n_sm / 2 : 1;
  double best = 0.0;
  int best_s = 1, best_a = 1;
  for (int a = 1; a <= (rows > NT ? 2 : 1); ++a) {
    const int tiles_n = (rows + a * NT - 1) / (a * NT);
    for (int s = 1; s <= max_splits && s <= (kb / 4 > 0 ? kb / 4 : 1); ++s) {
      const int per = (kb + s - 1) / s;
      if ((kb + per - 1) / per != s) continue;              // would leave an empty split
      if (fixed_splits > 0 && s != fixed_splits) continue;
      const int waves = (pairs * tiles_n * s + per_wave - 1) / per_wave;
      const double t_main = waves * (7500.0 + per * (a == 2 ? 1000.0 : 760.0) + a * 3000.0);
      const double t_slabs = (s - 1) * 2.0 * rows * static_cast<double>(n_out) * 4.0 / (30.0 * n_sm);
      const double t = t_main + t_slabs;
      if (best == 0.0 || t < best) { best = t; best_s = s; best_a = a; }
    }
  }
  *splits_out = best_s;
  *n_acc_out = best_a;
}

// Used for more than 128 token rows; every weight segment but the last must be whole 256-row pairs.
bool cod_gemm_tc2_supported(const cod_ctx* c, const GemmArgs& g) {
  if (c->cfg.dtype != COD_BF16 || g.a_rows != nullptr || g.rows_gate || g.n_rows <= 128) return false;
  if (g.K % 8 || g.lda % 8) return false;
  if ((reinterpret_cast<uintptr_t>(g.A) & 15u) != 0) return false;
  for (int i = 0; i < g.n_seg; ++i) {
    if ((reinterpret_cast<uintptr_t>(g.seg[i].B) & 15u) != 0) return false;
    if (i + 1 < g.n_seg && g.seg[i].N % (2 * BM)) return false;
  }
  return encode_fn() != nullptr;
}

int cod_launch_gemm_tc2(cod_ctx* c, const GemmArgs& g, cudaStream_t st) {
  Tc2Params p{};
  p.K = g.K;
  p.kb_total = (g.K + BK - 1) / BK;
  int splits = g.splits < 1 ? 1 : g.splits;
  p.kb_per_split = (p.kb_total + splits - 1) / splits;
  splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
  if (splits != g.splits) return COD_ERR_INVALID_ARG;
  p.n_rows = g.n_rows;
  p.n_rows_dev = g.n_rows_dev;
  p.group_split_dev = g.group_split_dev;
  if (g.group_split_dev && (g.n_seg != 2 || g.amax != nullptr || g.seg[0].N != g.seg[1].N)) return COD_ERR_INVALID_ARG;
  int pairs = 0;
  for (int i = 0; i < 3; ++i) {
    if (i < g.n_seg) {
      pairs += (g.seg[i].N + 2 * BM - 1) / (2 * BM);
      p.seg_N[i] = g.seg[i].N;
    }
    p.pair_end[i] = pairs;
  }
  p.n_seg = g.n_seg;
  p.n_acc = g.n_acc;
  if (p.n_acc != 1 && p.n_acc != 2) {
    int s_unused, n_out = 0;
    for (int i = 0; i < g.n_seg; ++i) n_out += g.seg[i].N;
    cod_plan_gemm_tc2(c->n_sm, n_out, g.K, g.n_rows, COD_MAX_SPLITS, splits, &s_unused, &p.n_acc);
  }
  p.stages = p.n_acc == 2 ? 4 : MAX_STAGES;
  p.n_tiles_n = (g.n_rows + p.n_acc * NT - 1) / (p.n_acc * NT);
  p.C = g.C;
  p.ldc = g.ldc;
  p.staged = (g.ldc % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.C) & 15u) == 0);
  for (int i = 0; i < g.n_seg; ++i) p.staged = p.staged && (g.seg[i].N % 4 == 0);
  p.amax = g.amax;
  p.lse_part = g.amax ? g.lse_part : nullptr;
  p.sample_state = g.sample_state;
  p.status = c->status;

  CUtensorMap mw[3], ma;
  for (int i = 0; i < 3; ++i) {
    const int j = i < g.n_seg ? i : 0;
    if (!make_map_2d(&mw[i], g.seg[j].B, g.seg[j].N, g.K, g.K, BM)) return COD_ERR_CUDA;
  }
  if (!make_map_2d(&ma, g.A, g.n_rows, g.K, g.lda, NT / 2)) return COD_ERR_CUDA;

  const size_t smem = static_cast<size_t>(p.stages) * (A_TILE_BYTES + p.n_acc * B_TILE_BYTES) + 1024 + 18 * 8 +
                      static_cast<size_t>(4) * p.n_acc * NT * 8;
  // the attribute belongs to (kernel, device): one record per device the process may use
  static size_t configured_dev[64][2] = {};
  size_t* configured = configured_dev[c->device & 63];
  const int sample = p.lse_part != nullptr ? 1 : 0;
  if (smem > configured[sample]) {
    const cudaError_t e = sample ? cudaFuncSetAttribute(k_gemm_tc2<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem))
                                 : cudaFuncSetAttribute(k_gemm_tc2<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return COD_ERR_CUDA;
    configured[sample] = smem;
  }
  // The argmax launches (no split-K, all rows in one two-accumulator tile) run in waves of one pair per two SMs; the
  // weight tiles beyond the last whole wave would hold two SMs each for a whole tile time while the rest idle
  // (151936 columns: 594 tiles = 8 waves of 74 + 2). Those tiles are launched as two pairs each, one accumulator
  // (256 token rows) per pair: half the time for the leftover wave.
  p.tail_pairs = 0;
  const int per_wave = c->n_sm / 2;
  if (g.amax != nullptr && splits == 1 && p.n_acc == 2 && p.n_tiles_n == 1 && per_wave > 0 && pairs > per_wave &&
      2 * (pairs % per_wave) <= per_wave)
    p.tail_pairs = pairs % per_wave;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2, (pairs + p.tail_pairs) * p.n_tiles_n, splits);
  cfg.blockDim = dim3(NTHREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = c->pdl ? 2 : 1;
  const cudaError_t le = sample ? cudaLaunchKernelEx(&cfg, k_gemm_tc2<true>, mw[0], mw[1], mw[2], ma, p)
                                : cudaLaunchKernelEx(&cfg, k_gemm_tc2<false>, mw[0], mw[1], mw[2], ma, p);
  if (le != cudaSuccess) return COD_ERR_CUDA;
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}
