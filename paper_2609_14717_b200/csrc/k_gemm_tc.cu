// Weight-streaming GEMM on the 5th-generation tensor cores (tcgen05), bf16 in / float out:
//   C[i, n] = sum_k A[i, k] * B[n, k]     A: activations [rows, K], B: weights [N, K].
//
// The operands are swapped for the MMA: the 128 weight rows of a tile are the MMA's M
// dimension and the (few) activation rows its N dimension (16..256), so a round with 16
// token rows wastes no tensor work and every CTA streams a disjoint slab of the weight
// matrix exactly once. Both tiles are staged K-major by TMA with the 128-byte swizzle into
// a multi-stage shared-memory ring; one elected thread issues tcgen05.mma, the accumulator
// lives in tensor memory (one lane per weight row, one column per token) and is read back
// with tcgen05.ld by four epilogue warps.
//
//   warp 0-3  epilogue (TMEM lanes 32*w .. 32*w+31)     warp 4  TMA producer     warp 5  MMA issuer
//
// Epilogues: float partial sums (split-K slabs, reduced by the row-wise kernels), or a fused
// per-token argmax over the weight rows for the LM head (logits are never stored).
// Every mbarrier wait is bounded: on expiry the CTA raises COD_DEV_TIMEOUT and leaves cleanly.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128;       // weight rows per CTA (MMA M)
constexpr int BK = 64;        // K elements per stage = one 128-byte swizzled row of bf16
constexpr int UK = 16;        // K elements per tcgen05.mma (kind::f16)
constexpr int NTHREADS = 192;
constexpr uint32_t A_TILE_BYTES = BM * BK * 2;   // 16 KB

struct TcParams {
  int K;
  int kb_total, kb_per_split;
  int n_rows;                 // rows (upper bound when n_rows_dev is set)
  const int* n_rows_dev;
  int rows_gate;              // n_rows_dev only gates: all rows if positive, none if zero
  int NT;                     // token rows per CTA = MMA N (multiple of 16, <= 256)
  int tmem_cols;              // power of two >= max(32, NT)
  int stages;
  int seg_tile_end[3];        // cumulative count of 128-row tiles after each weight segment
  int seg_N[3];
  int n_seg;
  int staged;                 // epilogue may transpose through shared memory (16-byte aligned feature runs)
  float* C;
  int ldc;
  unsigned long long* amax;
  const uint8_t* wt[3];       // per weight segment: tile-major copy (16 KB tiles), or null
  float2* lse_part;           // sampling form of the argmax epilogue (null: plain argmax)
  uint32_t sample_state;
  uint32_t* status;
  long long wait_limit;       // SM cycles a bounded wait may last
  int skip_copies;            // self-test of the failure path: the producer requests nothing, so the waits run out
  int pin_tiles;              // weight tiles [0, pin_tiles) of the launch are fetched evict-last (kept in L2 for the next round)
  // rank form (RANK kernels): per token row, how many weight rows score above a reference row
  const float* rank_ref;      // [n_rows] the reference row's logit
  const int32_t* rank_tok;    // [n_rows] the reference row's index (excluded from the count)
  unsigned int* rank_out;     // [n_rows] counts, zero before the launch
};

// AND of a predicate over the 128 threads of warps 0-3 (named barrier 1)
__device__ __forceinline__ bool bar_and_128(bool v) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(static_cast<uint32_t>(v)) : "memory");
  return r != 0;
}


// Weight tiles with an L2 eviction hint: a weight is read once per launch, so its lines should leave L2 first
// (evict-first) - except a prefix of one launch per round that fits L2 and is asked to stay (evict-last), so that
// the next round finds it there.
__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar), "l"(pol) : "memory");
}

// SAMPLE selects the sampling form of the argmax epilogue, WIDE the transposing store epilogue
// (32 token rows and more) and RANK the counting epilogue at compile time, so the kernel a batch-1
// round launches a dozen times carries none of them: with ~45 short kernels per round, instruction
// fetch of cold code shows.
template <bool SAMPLE, bool WIDE, bool RANK>
__global__ void __launch_bounds__(NTHREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
          const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_a, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle pattern
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t b_tile_bytes = static_cast<uint32_t>(p.NT) * BK * 2;
  const uint32_t stage_bytes = A_TILE_BYTES + b_tile_bytes;
  uint8_t* ctl = sm + static_cast<size_t>(p.stages) * stage_bytes;     // barriers and small state
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ctl);               // [stages]
  uint64_t* empty_bar = full_bar + 16;                                 // [stages]
  uint64_t* acc_bar = full_bar + 32;                                   // accumulator ready
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(full_bar + 33);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned long long* red = reinterpret_cast<unsigned long long*>(full_bar + 34);   // [4][NT] argmax keys, one row per epilogue warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tile = blockIdx.x, m_tile = blockIdx.y, split = blockIdx.z;
  const int i0 = n_tile * p.NT;

  // weight segment of this tile
  int sidx = 0;
  while (sidx < p.n_seg - 1 && m_tile >= p.seg_tile_end[sidx]) ++sidx;
  const int tile_in_seg = m_tile - (sidx ? p.seg_tile_end[sidx - 1] : 0);
  const int f0 = tile_in_seg * BM;                // first weight row within the segment
  int col0 = f0;                                  // first output column
  for (int s = 0; s < sidx; ++s) col0 += p.seg_N[s];
  const int seg_N = p.seg_N[sidx];
  const CUtensorMap* map_w = sidx == 0 ? &map_w0 : (sidx == 1 ? &map_w1 : &map_w2);
  // tile-major copy of this segment: tile (tile_in_seg, kb) is 16 KB at ((tile_in_seg * kb_total) + kb) * 16 KB
  const uint8_t* wt = p.wt[sidx] ? p.wt[sidx] + static_cast<size_t>(tile_in_seg) * p.kb_total * A_TILE_BYTES : nullptr;

  const int kb0 = split * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
  const int n_pre = min(p.stages, kb1 - kb0);     // stages whose weight tile is requested ahead of the dependency

  // ---- before the dependency on the previous kernel resolves: set up, and start streaming the
  // weights (nothing in the stream writes them) so the first stages are in flight or landed by the
  // time the activations exist. Their bytes are counted on the stage's barrier before its
  // expect_tx below, which the transaction count allows.
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(full_bar + s), 1); mbar_init(smem_u32(empty_bar + s), 1); }
    mbar_init(smem_u32(acc_bar), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int t = threadIdx.x; t < 4 * p.NT; t += NTHREADS) red[t] = 0ull;
  if (warp == 5) tmem_alloc(smem_u32(tmem_slot), static_cast<uint32_t>(p.tmem_cols));
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  uint64_t pol_w;
  if (m_tile < p.pin_tiles) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_w));
  else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_w));
  if (warp == 4 && lane == 0 && !p.skip_copies)
    for (int it = 0; it < n_pre; ++it)
      if (wt) bulk_load_hint(base + it * stage_bytes, wt + static_cast<size_t>(kb0 + it) * A_TILE_BYTES, A_TILE_BYTES, smem_u32(full_bar + it), pol_w);
      else tma_load_2d_hint(base + it * stage_bytes, map_w, (kb0 + it) * BK, f0, smem_u32(full_bar + it), pol_w);

  cod_pdl_prologue();
  const int n_rows = p.n_rows_dev ? (p.rows_gate ? (*p.n_rows_dev > 0 ? p.n_rows : 0) : min(*p.n_rows_dev, p.n_rows)) : p.n_rows;
  const int n_kb = i0 < n_rows ? kb1 - kb0 : 0;   // 0: no token rows here, only the requested weights to absorb

  if (warp == 4) {
    // ------------------------------------------------ TMA producer
    if (lane == 0 && !p.skip_copies) {
      if (n_kb == 0) {
        for (int it = 0; it < n_pre; ++it) {
          mbar_expect_tx(smem_u32(full_bar + it), A_TILE_BYTES);
          if (!mbar_wait(smem_u32(full_bar + it), 0, abort_flag, p.status, p.wait_limit)) break;
        }
      }
      for (int it = 0; it < n_kb; ++it) {
        const int s = it % p.stages, use = it / p.stages;
        if (use > 0 && !mbar_wait(smem_u32(empty_bar + s), (use - 1) & 1, abort_flag, p.status, p.wait_limit)) break;
        const uint32_t fb = smem_u32(full_bar + s);
        mbar_expect_tx(fb, stage_bytes);
        const uint32_t a_dst = base + s * stage_bytes;
        const int k = (kb0 + it) * BK;
        if (it >= n_pre) {
          if (wt) bulk_load_hint(a_dst, wt + static_cast<size_t>(kb0 + it) * A_TILE_BYTES, A_TILE_BYTES, fb, pol_w);
          else tma_load_2d_hint(a_dst, map_w, k, f0, fb, pol_w);
        }
        tma_load_2d(a_dst + A_TILE_BYTES, &map_a, k, i0, fb);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc(BM, p.NT, 0);
      bool ok = true;
      for (int it = 0; it < n_kb && ok; ++it) {
        const int s = it % p.stages, use = it / p.stages;
        ok = mbar_wait(smem_u32(full_bar + s), use & 1, abort_flag, p.status, p.wait_limit);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = base + s * stage_bytes;
        const uint64_t a_desc = desc_kmajor_sw128(a_addr), b_desc = desc_kmajor_sw128(a_addr + A_TILE_BYTES);
#pragma unroll
        for (int k = 0; k < BK / UK; ++k)       // advance 32 bytes (16 bf16) along K inside the swizzled row
          umma_bf16(tmem_base, a_desc + (k * UK * 2 >> 4), b_desc + (k * UK * 2 >> 4), idesc, (it | k) ? 1u : 0u);
        umma_commit(smem_u32(empty_bar + s));   // frees the stage when these MMAs retire
      }
      if (ok && n_kb > 0) umma_commit(smem_u32(acc_bar));
    }
  } else if (n_kb > 0) {
    // ------------------------------------------------ epilogue warps 0..3
    // one decision for the four epilogue warps (they meet at a named barrier below)
    const bool ok = bar_and_128(mbar_wait(smem_u32(acc_bar), 0, abort_flag, p.status, p.wait_limit));
    tc_fence_after();
    const int f = f0 + warp * 32 + lane;                    // weight row within the segment
    const bool f_ok = f < seg_N;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
    if (RANK) {
      // Per token column: how many of this warp's 32 weight rows lie above the column's reference
      // logit (ties: the lower index first; the reference row itself never counts). One ballot per
      // column, lane j keeps column c + j. References sit in the idle pipeline buffers.
      float* ref_v = reinterpret_cast<float*>(sm);
      int* ref_t = reinterpret_cast<int*>(sm + 1024);
      unsigned int* cnt = reinterpret_cast<unsigned int*>(red);
      for (int t = threadIdx.x; t < p.NT; t += 128) {
        const bool in = i0 + t < n_rows;
        ref_v[t] = in ? p.rank_ref[i0 + t] : INFINITY;
        ref_t[t] = in ? p.rank_tok[i0 + t] : -1;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      const int idx = col0 + warp * 32 + lane;
      for (int c = 0; c < p.NT && ok; c += 32) {
        uint32_t v[32];
        if (c + 32 <= p.NT) {
          tmem_ld32(t_lane + c, v);
        } else {                                   // NT is a multiple of 16: a last half chunk
          uint32_t h[16];
          tmem_ld16(t_lane + c, h);
#pragma unroll
          for (int j = 0; j < 16; ++j) { v[j] = h[j]; v[16 + j] = 0xFF800000u; }
        }
        unsigned int mine = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int cj = min(c + j, p.NT - 1);
          const float x = __uint_as_float(v[j]), rv = ref_v[cj];
          const int rt = ref_t[cj];
          const bool above = f_ok && c + j < p.NT && idx != rt && (x > rv || (x == rv && idx < rt));
          const unsigned int b = __ballot_sync(0xffffffffu, above);
          if (lane == j) mine = __popc(b);
        }
        if (c + lane < p.NT) cnt[warp * p.NT + c + lane] = mine;
      }
    } else if (WIDE && ok && p.amax == nullptr) {
      // The accumulator has features on lanes and tokens on columns; C wants a token's features
      // contiguous. Transpose 32 tokens at a time through the (now idle) pipeline buffers and store
      // whole 512-byte feature runs: two 16 KB buffers, one barrier of the four warps per chunk.
      float* C = p.C + static_cast<size_t>(split) * p.n_rows * p.ldc + col0;
      float* stage = reinterpret_cast<float*>(sm);
      const int f_left = seg_N - f0;                       // features of this tile that exist
      for (int c = 0, q = 0; c < p.NT && i0 + c < n_rows; c += 32, q ^= 1) {
        uint32_t v[32];
        if (c + 32 <= p.NT) {
          tmem_ld32(t_lane + c, v);
        } else {                                           // NT is a multiple of 16: a last half chunk
          uint32_t h[16];
          tmem_ld16(t_lane + c, h);
#pragma unroll
          for (int j = 0; j < 16; ++j) { v[j] = h[j]; v[16 + j] = 0u; }
        }
        float* buf = stage + q * (32 * BM);
#pragma unroll
        for (int j = 0; j < 32; ++j) buf[j * BM + warp * 32 + lane] = __uint_as_float(v[j]);
        asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const int tok = warp * 8 + t, i = i0 + c + tok;
          if (c + tok < p.NT && i < n_rows && lane * 4 < f_left)
            *reinterpret_cast<float4*>(C + static_cast<size_t>(i) * p.ldc + lane * 4) =
                *reinterpret_cast<const float4*>(buf + tok * BM + lane * 4);
        }
      }
    } else if (ok && p.amax == nullptr) {
      float* C = p.C + static_cast<size_t>(split) * p.n_rows * p.ldc;
      for (int c = 0; c < p.NT; c += 16) {
        uint32_t v[16];
        tmem_ld16(t_lane + c, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int i = i0 + c + j;
          if (f_ok && i < n_rows) C[static_cast<size_t>(i) * p.ldc + col0 + warp * 32 + lane] = __uint_as_float(v[j]);
        }
      }
    } else if (SAMPLE && ok) {
      // sampling form: Gumbel noise on every logit before the argmax, and soft-max partials per column.
      // Scratch in the idle pipeline buffers: row states, then per-warp (m, sum) of every column.
      uint32_t* hrow = reinterpret_cast<uint32_t*>(sm);
      float* red_m = reinterpret_cast<float*>(sm + 4096);
      float* red_s = red_m + 4 * 256;
      for (int t = threadIdx.x; t < 256; t += 128) hrow[t] = mix32(p.sample_state + static_cast<uint32_t>(i0 + t));
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int c = 0; c < p.NT; c += 32) {
        uint32_t v[32];
        if (c + 32 <= p.NT) {
          tmem_ld32(t_lane + c, v);
        } else {                                   // NT is a multiple of 16: a last half chunk
          uint32_t h[16];
          tmem_ld16(t_lane + c, h);
#pragma unroll
          for (int j = 0; j < 16; ++j) { v[j] = h[j]; v[16 + j] = 0xFF800000u; }   // -inf: never wins, adds nothing
        }
        unsigned long long best;
        float m_ref, s_sum;
        sample_chunk(v, f_ok, static_cast<uint32_t>(col0 + warp * 32 + lane), hrow + c, lane, best, m_ref, s_sum);
        if (c + lane < p.NT) {
          red[warp * p.NT + c + lane] = best;
          red_m[warp * 256 + c + lane] = m_ref;
          red_s[warp * 256 + c + lane] = s_sum;
        }
      }
    } else if (ok) {
      // per-token (max, lowest row) over this warp's 32 weight rows, 32 token columns at a time
      const unsigned long long low = static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<unsigned>(col0 + warp * 32 + lane));
      for (int c = 0; c < p.NT; c += 32) {
        unsigned long long k[32];
        if (c + 32 <= p.NT) {
          uint32_t v[32];
          tmem_ld32(t_lane + c, v);
#pragma unroll
          for (int j = 0; j < 32; ++j)
            k[j] = f_ok ? ((static_cast<unsigned long long>(order_key(__uint_as_float(v[j]))) << 32) | low) : 0ull;
        } else {                                   // NT is a multiple of 16: a last half chunk
          uint32_t v[16];
          tmem_ld16(t_lane + c, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            k[j] = f_ok ? ((static_cast<unsigned long long>(order_key(__uint_as_float(v[j]))) << 32) | low) : 0ull;
            k[16 + j] = 0ull;
          }
        }
        const unsigned long long best = warp_colmax32(k, lane);
        if (c + lane < p.NT) red[warp * p.NT + c + lane] = best;
      }
    }
  }

  // ---------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  else if (RANK) {
    if (n_kb > 0) {
      const unsigned int* cnt = reinterpret_cast<const unsigned int*>(red);
      for (int t = threadIdx.x; t < p.NT; t += NTHREADS) {
        const unsigned int total = cnt[t] + cnt[p.NT + t] + cnt[2 * p.NT + t] + cnt[3 * p.NT + t];
        if (i0 + t < n_rows && total) atomicAdd(p.rank_out + i0 + t, total);
      }
    }
  }
  else if (p.amax != nullptr && n_kb > 0) {
    // the four epilogue warps merged their per-token keys in shared memory: one atomic per token
    for (int t = threadIdx.x; t < p.NT; t += NTHREADS) {
      if (i0 + t < n_rows) {
        unsigned long long best = red[t];
#pragma unroll
        for (int w = 1; w < 4; ++w) best = red[w * p.NT + t] > best ? red[w * p.NT + t] : best;
        atomicMax(p.amax + i0 + t, best);
        if (SAMPLE) {                                  // this tile's soft-max partial of token row i0 + t
          const float* red_m = reinterpret_cast<const float*>(sm + 4096);
          const float* red_s = red_m + 4 * 256;
          float m = red_m[t];
#pragma unroll
          for (int w = 1; w < 4; ++w) m = fmaxf(m, red_m[w * 256 + t]);
          float sum = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w)
            if (red_m[w * 256 + t] > -INFINITY) sum += red_s[w * 256 + t] * __expf(red_m[w * 256 + t] - m);
          p.lse_part[static_cast<size_t>(col0 / BM) * p.n_rows + i0 + t] = make_float2(m, sum);
        }
      }
    }
  }
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
  }
}

// ------------------------------------------------------------------ host side


}  // namespace

bool cod_gemm_tc_supported(const cod_ctx* c, const GemmArgs& g) {
  if (c->cfg.dtype != COD_BF16 || g.a_rows != nullptr || g.group_split_dev != nullptr) return false;
  if (g.K % 8 || g.lda % 8 || g.n_rows < 1) return false;
  if ((reinterpret_cast<uintptr_t>(g.A) & 15u) != 0) return false;
  for (int i = 0; i < g.n_seg; ++i) {
    if ((reinterpret_cast<uintptr_t>(g.seg[i].B) & 15u) != 0) return false;
    if (i + 1 < g.n_seg && g.seg[i].N % BM) return false;     // a tile must not straddle two matrices
  }
  return encode_fn() != nullptr;
}

int cod_launch_gemm_tc(cod_ctx* c, const GemmArgs& g, cudaStream_t st) {
  TcParams p{};
  p.K = g.K;
  p.kb_total = (g.K + BK - 1) / BK;
  int splits = g.splits < 1 ? 1 : g.splits;
  p.kb_per_split = (p.kb_total + splits - 1) / splits;
  splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;     // no empty split
  if (splits != g.splits) return COD_ERR_INVALID_ARG;               // the caller sized the partial slabs
  p.n_rows = g.n_rows;
  p.n_rows_dev = g.n_rows_dev;
  p.rows_gate = g.rows_gate;
  const int r16 = (g.n_rows + 15) / 16 * 16;
  p.NT = r16 < 256 ? r16 : 256;
  int cols = 32;
  while (cols < p.NT) cols <<= 1;
  p.tmem_cols = cols;
  const uint32_t stage_bytes = A_TILE_BYTES + static_cast<uint32_t>(p.NT) * BK * 2;
  int stages = static_cast<int>((200u * 1024u) / stage_bytes);
  if (stages > 8) stages = 8;
  // small tiles: leave room for two CTAs per SM - three when the grid is several waves deep (the LM head
  // at batch 1: 1187 CTAs), where a third resident CTA covers the other two's fill and drain bubbles
  // (203 -> 191 us); shallower grids keep the deeper ring, each CTA being alone on its share of an SM
  if (p.NT <= 32) {
    int tiles_all = 0;
    for (int i = 0; i < g.n_seg; ++i) tiles_all += (g.seg[i].N + BM - 1) / BM;
    const int cap = static_cast<long long>(tiles_all) * splits >= 3ll * c->n_sm ? 4 : 5;
    if (stages > cap) stages = cap;
  }
  if (stages > p.kb_per_split) stages = p.kb_per_split;
  if (stages < 1) stages = 1;
  p.stages = stages;
  int tiles = 0;
  for (int i = 0; i < 3; ++i) {
    if (i < g.n_seg) {
      tiles += (g.seg[i].N + BM - 1) / BM;
      p.seg_N[i] = g.seg[i].N;
    }
    p.seg_tile_end[i] = tiles;
  }
  p.n_seg = g.n_seg;
  p.C = g.C;
  p.ldc = g.ldc;
  p.staged = (g.ldc % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.C) & 15u) == 0) &&
             static_cast<size_t>(stages) * stage_bytes >= 2u * 32u * BM * sizeof(float);
  for (int i = 0; i < g.n_seg; ++i) p.staged = p.staged && (g.seg[i].N % 4 == 0);
  p.amax = g.amax;
  for (int i = 0; i < 3; ++i) p.wt[i] = i < g.n_seg ? static_cast<const uint8_t*>(g.seg[i].Bt) : nullptr;
  p.lse_part = g.amax ? g.lse_part : nullptr;
  p.sample_state = g.sample_state;
  p.status = c->status;
  p.wait_limit = c->wait_limit > 0 ? c->wait_limit : WAIT_LIMIT_CYCLES;
  p.skip_copies = c->selftest_skip_copies;
  // The round's first weight stream (the fc projection) keeps a prefix of its tiles in L2 for the next round: every
  // other stream of the round is evict-first, so about a third of the 126 MB survives a round (measured at batch 1:
  // 40-64 MB kept -> 410 -> 405 us per round; 96 MB -> no gain, the prefix then evicts itself).
  p.pin_tiles = g.klass == COD_K_FC ? static_cast<int>(COD_L2_KEEP_BYTES / (static_cast<long long>(g.K) * BM * 2)) : 0;

  CUtensorMap mw[3], ma;
  for (int i = 0; i < 3; ++i) {
    const int j = i < g.n_seg ? i : 0;
    if (!make_map_2d(&mw[i], g.seg[j].B, g.seg[j].N, g.K, g.K, BM)) return COD_ERR_CUDA;
  }
  if (!make_map_2d(&ma, g.A, g.n_rows, g.K, g.lda, p.NT)) return COD_ERR_CUDA;

  const size_t smem = static_cast<size_t>(stages) * stage_bytes + 1024 /* alignment slack */ + 34 * 8 + 4 * p.NT * 8;
  // four instantiations: plain (narrow store or argmax), wide store, sampling argmax, rank count
  const bool rank = g.rank_out != nullptr;
  if (rank) {
    if (g.amax != nullptr || g.rank_ref == nullptr || g.rank_tok == nullptr) return COD_ERR_INVALID_ARG;
    p.rank_ref = g.rank_ref; p.rank_tok = g.rank_tok; p.rank_out = g.rank_out;
  }
  const int variant = rank ? 3 : (p.lse_part != nullptr ? 2 : ((p.amax == nullptr && p.staged && p.NT >= 32) ? 1 : 0));
  using kernel_t = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const TcParams);
  static const kernel_t kernels[4] = {k_gemm_tc<false, false, false>, k_gemm_tc<false, true, false>,
                                      k_gemm_tc<true, false, false>, k_gemm_tc<false, false, true>};
  // the attribute belongs to (kernel, device): one record per device the process may use
  static size_t configured_dev[64][4] = {};
  size_t* configured = configured_dev[c->device & 63];
  if (smem > configured[variant]) {
    if (cudaFuncSetAttribute(kernels[variant], cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
      return COD_ERR_CUDA;
    configured[variant] = smem;
  }
  dim3 grid((g.n_rows + p.NT - 1) / p.NT, tiles, splits);
  cod_launch_pdl(c, kernels[variant], grid, NTHREADS, smem, st, mw[0], mw[1], mw[2], ma, p);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

// ------------------------------------------------------------------ read-out of the sampling head
// One warp per token row: merges the per-tile soft-max partials (m_t, s_t) into the log-sum-exp,
// takes the winning (perturbed logit, index) key, removes the winner's noise again (it is a pure
// function of seed, step, row and index) and reports q = exp(logit - lse).
namespace {
__global__ void k_finalize_sample(const unsigned long long* __restrict__ amax, const float2* __restrict__ lse_part,
                                  int n_tiles, int R, uint32_t state, int32_t* __restrict__ tok,
                                  float* __restrict__ q_tok, float* __restrict__ lse_out, int W,
                                  const int32_t* __restrict__ bonus, int32_t* __restrict__ next_draft) {
  cod_pdl_prologue();
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= R) return;
  float m = -INFINITY, s = 0.f;
  for (int t = lane; t < n_tiles; t += 32) {
    const float2 ms = lse_part[static_cast<size_t>(t) * R + r];
    if (ms.x > -INFINITY) {
      const float mn = fmaxf(m, ms.x);
      s = s * __expf(m - mn) + ms.y * __expf(ms.x - mn);      // exp(-inf) = 0 covers the first term
      m = mn;
    }
  }
  for (int o = 16; o >= 1; o >>= 1) {
    const float mo = __shfl_xor_sync(0xffffffffu, m, o), so = __shfl_xor_sync(0xffffffffu, s, o);
    const float mn = fmaxf(m, mo);
    if (mn > -INFINITY) s = s * __expf(m - mn) + so * __expf(mo - mn);
    m = mn;
  }
  if (lane == 0) {
    const unsigned long long key = amax[r];
    const int idx = cod_unpack_index(key);
    const float pert = tc::order_key_to_float(static_cast<unsigned>(key >> 32));
    const float raw = pert - tc::gumbel_noise(tc::mix32(state + static_cast<uint32_t>(r)), static_cast<uint32_t>(idx));
    const float lse = m + logf(s);
    if (tok) tok[r] = idx;
    if (q_tok) q_tok[r] = expf(raw - lse);
    if (lse_out) lse_out[r] = lse;
    if (next_draft) next_draft[r] = (r % W == 0) ? bonus[r / W] : idx;     // row 0 of a block is the bonus token
  }
}
}  // namespace

int cod_launch_finalize_sample(cod_ctx* c, int R, uint32_t state, int32_t* tok, float* q_tok, float* lse,
                               cudaStream_t st, const int32_t* bonus, int32_t* next_draft) {
  ProfScope prof(c, COD_K_ROWOPS, st);
  const int n_tiles = (c->cfg.vocab + BM - 1) / BM;
  cod_launch_pdl(c, k_finalize_sample, (R + 3) / 4, 128, 0, st, c->amax, c->lse_part, n_tiles, R, state, tok, q_tok, lse, c->cfg.block,
                 bonus, next_draft);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}
uint32_t cod_sample_state(unsigned long long seed, uint32_t step) { return tc::sample_state(seed, step); }

// ------------------------------------------------------------------ tile-major weight copy
namespace {
__global__ void k_retile(const __nv_bfloat16* __restrict__ B, int N, int K, uint8_t* __restrict__ Bt) {
  const int kb = blockIdx.x, tile = blockIdx.y, kb_total = gridDim.x;
  uint4* dst = reinterpret_cast<uint4*>(Bt + (static_cast<size_t>(tile) * kb_total + kb) * A_TILE_BYTES);
  for (int idx = threadIdx.x; idx < BM * 8; idx += blockDim.x) {        // 16-byte chunks: 128 rows x 8
    const int r = idx >> 3, ch = idx & 7;
    const int row = tile * BM + r, col = kb * BK + ch * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < N && col < K) v = *reinterpret_cast<const uint4*>(B + static_cast<size_t>(row) * K + col);   // K % 8 == 0
    dst[r * 8 + (ch ^ (r & 7))] = v;                                       // the 128-byte swizzle
  }
}
}  // namespace

size_t cod_retile_bytes(int N, int K) {
  return static_cast<size_t>((N + BM - 1) / BM) * ((K + BK - 1) / BK) * A_TILE_BYTES;
}

int cod_launch_retile(cod_ctx* c, const void* B, int N, int K, void* Bt, cudaStream_t st) {
  if (K % 8) return COD_ERR_UNSUPPORTED;
  const dim3 grid((K + BK - 1) / BK, (N + BM - 1) / BM);
  k_retile<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(B), N, K, static_cast<uint8_t*>(Bt));
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

