// Part 4 on the tensor cores: split-KV block attention over [C_l; U_l; block] for bf16, head
// size 128, page size 16 (Section 2 "Preliminaries"; Algorithm 1 "the next draft reads ctx_l").
//
// A CTA owns one (sequence, KV head, split). The W * (n_q / n_kv) query rows that share the KV
// head are the MMA's M dimension, so every K/V byte is read once per sequence.
//   S = Q K^T   tcgen05.mma, Q and the K tile K-major in shared memory, S in tensor memory
//   P = exp2(S * c - m)   one thread per query row: row max and row sum are thread-local
//   O = P V     tcgen05.mma, P (bf16) K-major in shared memory, the V tile MN-major
// With 64 query rows (block 16, GQA 4) an M = 64 accumulator uses lanes 0-15 of each 32-lane
// quarter of tensor memory; a second, independent M = 64 tile is placed on lanes 16-31, so the
// CTA works on two 64-key tiles at once and all 128 softmax threads have a row. With 128 query
// rows (block 32) one M = 128 tile is used.
//
// Keys: [0, F) with F = 16 * floor(L / 16) come from whole pages, fetched by TMA straight from the
// block table into a shared-memory ring (two 16 x 64-element boxes per page and operand, no
// multi-destination loads). The remaining L - F committed rows, the c carried rows and the W
// block rows form the tail, gathered with plain 128-bit loads by one extra CTA per (sequence, head)
// which zero-fills the padding, so stale or unallocated rows are never read.
// Each 64-key tile yields an unnormalised partial (o, m, l); a second kernel merges them.
//
//   warps 0-3 softmax / accumulation     warp 4 TMA producer     warp 5 MMA issuer
// Every mbarrier wait is bounded and raises COD_DEV_TIMEOUT instead of spinning forever.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int HD = 128, PAGE = 16, KT = 64;           // head size, page size, keys per tile
constexpr int NTHREADS = 224;     // 4 softmax warps, K producer, MMA issuer, V producer
constexpr uint32_t TILE_BYTES = KT * HD * 2;           // one 64-key K or V tile: 16 KB
constexpr uint32_t HALF_BYTES = KT * 128;              // 64 keys x 64 elements: 8 KB

struct AttnParams {
  const __nv_bfloat16 *q, *kb, *vb;     // rotated q [R, n_q*hd]; rotated k_blk, v_blk [R, n_kv*hd]
  const __nv_bfloat16 *pool, *carry;
  const int *block_table, *committed_len, *carry_len;
  int use_carry, layer, W, rep, n_kv, n_pages, max_pages, max_batch;
  int cap;                              // rows of a carry slot (retention rounds * W)
  int split_len;                        // keys of the paged region per CTA (multiple of 128)
  int max_parts;                        // partial slots per (sequence, KV head)
  float* part_o;                        // [S][n_kv][max_parts][M][hd]
  float* part_ml;                       // [S][n_kv][max_parts][M][4]   m (natural log units), l, l_carry
  const int* order;                     // null: CTA (x, y, z) = (part, head, sequence). Else CTA (x, y) = (head, i) works
                                        // on part order[i] = sequence << 16 | part, longest first; -1: nothing
  int run_ahead;                // the launch's stream predecessor writes only q / k_blk / v_blk (see k_attn_tc)
  int n_list;                           // entries of order[] (persistent kernel)
  int* work_counter;                    // persistent kernel: units taken beyond each CTA's first (zero before the launch)
  uint32_t* status;
};


// L2 eviction hints. The K/V stream is read once per call: marked evict-first it does not push out what the call
// itself will read again (the partial results written below, marked evict-last, which the merge kernel reads).
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void st_float4_hint(float4* ptr, float a, float b, float c, float d, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(ptr), "f"(a), "f"(b), "f"(c), "f"(d), "l"(pol) : "memory");
}

// One query row's 64 scores -> probabilities exp2(s * sl2 + neg), stored as bf16 into the row of the P tile
// (16-byte chunks XOR-swizzled by the row) and summed. TAIL: also the mass on the carried keys [car0, car0 + c)
// (only tail tiles hold carried keys; the common tile carries none of that bookkeeping).
template <bool TAIL>
__device__ __forceinline__ void softmax_store(const float (&sc)[64], float sl2, float neg, uint8_t* prow, int r, int car0,
                                              int c, float& psum, float& pcar) {
  float ps4[4] = {0.f, 0.f, 0.f, 0.f};
  pcar = 0.f;
#pragma unroll
  for (int ch = 0; ch < 8; ++ch) {
    uint32_t packed[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int j = ch * 8 + e * 2;
      const float p0 = tc::ex2_approx(fmaf(sc[j], sl2, neg)), p1 = tc::ex2_approx(fmaf(sc[j + 1], sl2, neg));
      ps4[e] += p0 + p1;
      if (TAIL) {
        if (j >= car0 && j < car0 + c) pcar += p0;
        if (j + 1 >= car0 && j + 1 < car0 + c) pcar += p1;
      }
      const __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
      packed[e] = *reinterpret_cast<const uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(prow + ((ch ^ (r & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  }
  psum = (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
}

template <bool DUAL>
struct Geo {
  static constexpr int TILES = DUAL ? 2 : 1;             // 64-key tiles per iteration
  static constexpr int MROWS = DUAL ? 64 : 128;          // MMA M
  static constexpr int KEYS_IT = KT * TILES;
  static constexpr int NK = DUAL ? 1 : 2;                // K ring slots
  static constexpr int NV = 1;                           // V ring slots (two CTAs fit on an SM either way)
  static constexpr uint32_t SLOT = TILE_BYTES * TILES;
  static constexpr uint32_t Q_BYTES = MROWS * HD * 2;
  static constexpr uint32_t Q_HALF = MROWS * 128;
  static constexpr uint32_t P_TILE = MROWS * 128;        // [MROWS][64 keys] bf16
  static constexpr uint32_t P_BUF = P_TILE * TILES;
  static constexpr uint32_t OFF_P = Q_BYTES;
  static constexpr uint32_t OFF_K = OFF_P + P_BUF;       // P is single-buffered
  static constexpr uint32_t OFF_V = OFF_K + NK * SLOT;
  static constexpr uint32_t OFF_CTL = OFF_V + NV * SLOT;
  static constexpr uint32_t SMEM = OFF_CTL + 512 + 1024 + 1024;   // barriers and the unit ring, page ids, alignment slack
  // tensor memory columns: S[2] (64 each) then O (128)
  static constexpr uint32_t COL_S = 0, COL_O = 128, TMEM_COLS = 256;
};

template <bool DUAL>
__global__ void __launch_bounds__(NTHREADS, 2)
k_attn_tc(const __grid_constant__ CUtensorMap map_pool, const __grid_constant__ CUtensorMap map_zero, const AttnParams p) {
  // Small grids (no work list) run ahead of the dependency: barriers, tensor memory, page ids and the paged K/V
  // stream touch nothing the previous kernel of the stream writes (it produces q, k_blk, v_blk or the work list;
  // everything older has completed before this grid may start), so only the warps that read those wait for it.
  const bool early = p.order == nullptr && p.run_ahead;
  if (!early) cod_pdl_prologue();
  using G = Geo<DUAL>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + G::OFF_CTL);
  uint64_t* k_full = bars;                  // [NK]
  uint64_t* k_empty = bars + 5;             // [NK]
  uint64_t* v_full = bars + 10;             // [NV]
  uint64_t* v_empty = bars + 15;            // [NV]
  uint64_t* s_full = bars + 20;             // [2]
  uint64_t* p_full = bars + 22;             // [2]
  uint64_t* o_full = bars + 24;             // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
  uint64_t* q_ready = bars + 27;            // the Q tile is in shared memory
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* page_ids = reinterpret_cast<int*>(bars + 28);       // [split_len / 16] <= 256 entries

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int split = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
  if (p.order != nullptr) {
    const int item = p.order[blockIdx.y];
    if (item < 0) return;
    h = blockIdx.x; s = item >> 16; split = item & 0xFFFF;
  }
  const int M = p.W * p.rep;

  uint32_t flags = 0;
  int L = p.committed_len[s];
  int c = p.use_carry ? p.carry_len[s] : 0;
  if (L < 0 || L > p.max_pages * PAGE) { flags |= COD_DEV_BAD_LEN; L = max(0, min(L, p.max_pages * PAGE)); }
  if (c < 0 || c > p.cap) { flags |= COD_DEV_BAD_LEN; c = max(0, min(c, p.cap)); }
  const int F = (L / PAGE) * PAGE;                       // keys held in whole pages
  const int n_reg = (F + p.split_len - 1) / p.split_len; // CTAs over the paged region
  if (split > n_reg) return;
  const bool is_tail = split == n_reg;
  const int Lr = L - F;                                  // committed rows in the last, partial page
  const int n_tail = Lr + c + p.W;
  const int k_begin = is_tail ? 0 : split * p.split_len;
  const int k_end = is_tail ? n_tail : min(F, k_begin + p.split_len);
  const int n_it = (k_end - k_begin + G::KEYS_IT - 1) / G::KEYS_IT;

  if (threadIdx.x == 0) {
    for (int i = 0; i < G::NK; ++i) { mbar_init(smem_u32(k_full + i), is_tail ? 128 : 1); mbar_init(smem_u32(k_empty + i), 1); }
    for (int i = 0; i < G::NV; ++i) { mbar_init(smem_u32(v_full + i), is_tail ? 128 : 1); mbar_init(smem_u32(v_empty + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(s_full + i), 1); mbar_init(smem_u32(p_full + i), 128); mbar_init(smem_u32(o_full + i), 1); }
    mbar_init(smem_u32(q_ready), 128);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(smem_u32(tmem_slot), G::TMEM_COLS);
  if (warp == 4 && !is_tail) {
    // physical page of every logical page this CTA will touch, fetched once
    for (int i = lane; i < (k_end - k_begin + PAGE - 1) / PAGE; i += 32) {
      int pg = p.block_table[s * p.max_pages + k_begin / PAGE + i];
      if (pg < 0 || pg >= p.n_pages) { flags |= COD_DEV_BAD_PAGE; pg = -1; }
      page_ids[i] = pg;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Q tile: [half][row][64 elements], 128-byte rows, chunks of 16 bytes XOR-swizzled by (row & 7);
  // rows beyond the real query rows are zero.
  if (warp < 4) {
    if (early) cod_pdl_prologue();
    const int qw = p.n_kv * p.rep * HD;
    constexpr int QB = 8;                                   // independent 16-byte loads in flight per thread
    for (int idx0 = threadIdx.x; idx0 < G::MROWS * 16; idx0 += 128 * QB) {
      uint4 v[QB];
#pragma unroll
      for (int u = 0; u < QB; ++u) {
        const int idx = idx0 + u * 128, r = idx >> 4, ch = idx & 15;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (r < M) {
          const int i = r / p.rep, gg = r - i * p.rep;
          v[u] = *reinterpret_cast<const uint4*>(p.q + static_cast<size_t>(s * p.W + i) * qw + (h * p.rep + gg) * HD + ch * 8);
        }
      }
#pragma unroll
      for (int u = 0; u < QB; ++u) {
        const int idx = idx0 + u * 128, r = idx >> 4, ch = idx & 15;
        *reinterpret_cast<uint4*>(sm + (ch >> 3) * G::Q_HALF + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = v[u];
      }
    }
    fence_async_smem();
    mbar_arrive(smem_u32(q_ready));
  }

  if (warp == 4 || warp == 6) {
    // ------------------------------------------------ TMA producers (paged region only): warp 4 streams
    // the K tiles, warp 6 the V tiles, so the two rings are fed independently
    if (!is_tail) {
      const bool is_v = warp == 6;
      const int pages_it = G::KEYS_IT / PAGE;           // 8 or 4 pages per iteration, one per lane
      const int ring = is_v ? G::NV : G::NK;
      uint64_t* full = is_v ? v_full : k_full;
      uint64_t* empty = is_v ? v_empty : k_empty;
      const uint32_t ring_off = is_v ? G::OFF_V : G::OFF_K;
      const uint64_t pol_stream = l2_policy_evict_first();
      bool ok = true;
      for (int it = 0; it < n_it && ok; ++it) {
        const int key0 = k_begin + it * G::KEYS_IT + lane * PAGE;
        int row = -1;                                   // first row of this lane's page tile in the pool map
        if (lane < pages_it && key0 < k_end) {
          const int pg = page_ids[(key0 - k_begin) / PAGE];
          if (pg >= 0) row = (((p.layer * p.n_pages + pg) * p.n_kv + h) * 2 + (is_v ? 1 : 0)) * PAGE;
        }
        const uint32_t in_slot = (lane / (KT / PAGE)) * TILE_BYTES + (lane % (KT / PAGE)) * (PAGE * 128);
        const int slot = it % ring, use = it / ring;
        if (lane == 0 && use > 0) ok = mbar_wait(smem_u32(empty + slot), (use - 1) & 1, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        const uint32_t fb = smem_u32(full + slot);
        if (lane == 0) mbar_expect_tx(fb, G::SLOT);
        __syncwarp();
        if (lane < pages_it) {
          const uint32_t dst = base + ring_off + slot * G::SLOT + in_slot;
          if (row >= 0) {
            tma_load_3d_hint(dst, &map_pool, 0, 0, row, fb, pol_stream);
            tma_load_3d_hint(dst + HALF_BYTES, &map_pool, 0, 1, row, fb, pol_stream);
          } else {
            tma_load_3d(dst, &map_zero, 0, 0, 0, fb);
            tma_load_3d(dst + HALF_BYTES, &map_zero, 0, 1, 0, fb);
          }
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0 && n_it > 0) {
      const uint32_t idesc_qk = instr_desc(G::MROWS, KT, 0);
      const uint32_t idesc_pv = instr_desc(G::MROWS, HD, 1);
      const uint64_t q_desc = desc_kmajor_sw128(base);
      bool ok = true;
      auto issue_qk = [&](int it) -> bool {
        const int slot = it % G::NK;
        if (!mbar_wait(smem_u32(k_full + slot), (it / G::NK) & 1, abort_flag, p.status)) return false;
        tc_fence_after();
#pragma unroll
        for (int t = 0; t < G::TILES; ++t) {
          const uint64_t k_desc = desc_kmajor_sw128(base + G::OFF_K + slot * G::SLOT + t * TILE_BYTES);
          const uint32_t d = tmem_base + G::COL_S + (it & 1) * KT + (static_cast<uint32_t>(16 * t) << 16);
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint32_t qa = (k < 4 ? 0u : (G::Q_HALF >> 4)) + (k & 3) * 2;
            const uint32_t ka = (k < 4 ? 0u : (HALF_BYTES >> 4)) + (k & 3) * 2;
            umma_bf16(d, q_desc + qa, k_desc + ka, idesc_qk, k ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(s_full + (it & 1)));
        umma_commit(smem_u32(k_empty + slot));
        return true;
      };
      ok = mbar_wait(smem_u32(q_ready), 0, abort_flag, p.status) && issue_qk(0);
      for (int it = 0; it < n_it && ok; ++it) {
        if (it + 1 < n_it) ok = issue_qk(it + 1);
        if (!ok) break;
        const int slot = it % G::NV;
        ok = mbar_wait(smem_u32(p_full + (it & 1)), (it >> 1) & 1, abort_flag, p.status) &&
             mbar_wait(smem_u32(v_full + slot), (it / G::NV) & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int t = 0; t < G::TILES; ++t) {
          const uint64_t p_desc = desc_kmajor_sw128(base + G::OFF_P + t * G::P_TILE);
          const uint64_t v_desc = desc_mnmajor_sw128(base + G::OFF_V + slot * G::SLOT + t * TILE_BYTES, HALF_BYTES);
          const uint32_t d = tmem_base + G::COL_O + (static_cast<uint32_t>(16 * t) << 16);
#pragma unroll
          for (int kk = 0; kk < KT / 16; ++kk)       // 16 keys per MMA: 32 bytes along P's rows, 16 rows of V
            umma_bf16(d, p_desc + kk * 2, v_desc + kk * ((16 * 128) >> 4), idesc_pv, (it | kk) ? 1u : 0u);
        }
        umma_commit(smem_u32(o_full + (it & 1)));
        umma_commit(smem_u32(v_empty + slot));
      }
    }
  } else {
    // ------------------------------------------------ softmax: one thread per (row, tile)
    // O = sum_j p_j v_j accumulates in tensor memory across iterations, relative to a per-row
    // reference maximum m_ref. The reference only moves when the row maximum grows by more than
    // 2^8 in probability terms (then this warp rescales its rows of O in tensor memory), so the
    // common iteration touches S only: load scores, exponentiate, store P.
    const int T = threadIdx.x;
    const int tile = DUAL ? (lane >> 4) : 0;
    const int r = DUAL ? (16 * warp + (lane & 15)) : T;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(32 * warp) << 16);
    const float sl2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;   // raw score -> log2 units
    const float rescale_gap = 8.f / sl2;
    float m_ref = -INFINITY, l_run = 0.f, lc_run = 0.f;
    bool ok = true;

    for (int it = 0; it < n_it && ok; ++it) {
      if (is_tail) {
        // gather this iteration's rows (partial page, carried rows, block rows) with plain loads:
        // first the K rows (the MMA warp asks for them first), then the V rows. A ring slot that was
        // used before is taken only once the MMAs that read it have retired.
        constexpr int GB = 8;                               // independent 16-byte loads in flight per thread
#pragma unroll 1
        for (int kv = 0; kv < 2; ++kv) {
          const int ring = kv ? G::NV : G::NK;
          const int slot = it % ring, use = it / ring;
          uint64_t* full = kv ? v_full : k_full;
          uint64_t* empty = kv ? v_empty : k_empty;
          if (use > 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(empty + slot), (use - 1) & 1, abort_flag, p.status));
            if (!ok) break;
          }
          for (int idx0 = T; idx0 < G::KEYS_IT * 16; idx0 += 128 * GB) {
            uint4 val[GB];
            uint32_t dst[GB];
#pragma unroll
            for (int u = 0; u < GB; ++u) {
              const int idx = idx0 + u * 128;
              const int ch = idx & 15, j = idx >> 4;                          // chunk, key within iteration
              const int g = it * G::KEYS_IT + j;
              const __nv_bfloat16* src = nullptr;
              if (g < Lr) {
                int pg = p.block_table[s * p.max_pages + F / PAGE];
                if (pg < 0 || pg >= p.n_pages) { flags |= COD_DEV_BAD_PAGE; }
                else src = p.pool + ((((static_cast<size_t>(p.layer) * p.n_pages + pg) * p.n_kv + h) * 2 + kv) * PAGE + g) * HD;
              } else if (g < Lr + c) {
                src = p.carry + ((((static_cast<size_t>(p.layer) * p.max_batch + s) * p.n_kv + h) * 2 + kv) * p.cap + (g - Lr)) * HD;
              } else if (g < n_tail) {
                src = (kv ? p.vb : p.kb) + static_cast<size_t>(s * p.W + (g - Lr - c)) * (p.n_kv * HD) + h * HD;
              }
              val[u] = src ? *reinterpret_cast<const uint4*>(src + ch * 8) : make_uint4(0u, 0u, 0u, 0u);
              const int jj = j & (KT - 1), tl = j / KT;
              dst[u] = (kv ? G::OFF_V : G::OFF_K) + slot * G::SLOT + tl * TILE_BYTES +
                       (ch >> 3) * HALF_BYTES + jj * 128 + (((ch & 7) ^ (jj & 7)) << 4);
            }
#pragma unroll
            for (int u = 0; u < GB; ++u) *reinterpret_cast<uint4*>(sm + dst[u]) = val[u];
          }
          fence_async_smem();
          mbar_arrive(smem_u32(full + slot));
        }
        if (!ok) break;
      }

      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(s_full + (it & 1)), (it >> 1) & 1, abort_flag, p.status));
      if (!ok) break;
      tc_fence_after();
      const int key_t0 = k_begin + it * G::KEYS_IT + tile * KT;         // first key of this thread's tile
      const int n_valid = max(0, min(KT, k_end - key_t0));
      float sc[KT];
      {
        uint32_t v[32];
        tmem_ld32(t_lane + G::COL_S + (it & 1) * KT, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) sc[j] = __uint_as_float(v[j]);
        tmem_ld32(t_lane + G::COL_S + (it & 1) * KT + 32, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) sc[32 + j] = __uint_as_float(v[j]);
      }
      if (n_valid < KT) {                                  // only the last iteration of a split is ragged
#pragma unroll
        for (int j = 0; j < KT; ++j) sc[j] = j < n_valid ? sc[j] : -INFINITY;
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};      // four independent chains
#pragma unroll
      for (int j = 0; j < KT; j += 4) {
        mx4[0] = fmaxf(mx4[0], sc[j]); mx4[1] = fmaxf(mx4[1], sc[j + 1]);
        mx4[2] = fmaxf(mx4[2], sc[j + 2]); mx4[3] = fmaxf(mx4[3], sc[j + 3]);
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const bool need = mx > m_ref + rescale_gap;        // also true for the first finite maximum
      if (__any_sync(0xffffffffu, need)) {
        const float m_new = need ? mx : m_ref;
        const float factor = need ? ex2_approx((m_ref - m_new) * sl2) : 1.f;     // ex2(-inf) = 0
        if (it > 0) {
          // O is relative to the old reference: once PV(it-1) has landed, scale this warp's rows
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(o_full + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag, p.status));
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int q4 = 0; q4 < HD / 32; ++q4) {
            uint32_t v[32];
            tmem_ld32(t_lane + G::COL_O + q4 * 32, v);
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * factor);
            tmem_st32(t_lane + G::COL_O + q4 * 32, v);
          }
        }
        l_run *= factor;
        lc_run *= factor;
        m_ref = m_new;
      }
      if (it >= 1) {   // the P buffer about to be overwritten was read by PV(it-1)
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(o_full + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag, p.status));
        if (!ok) break;
      }
      const float neg = m_ref == -INFINITY ? 0.f : -m_ref * sl2;
      float psum, pcar;
      uint8_t* prow = sm + G::OFF_P + tile * G::P_TILE + r * 128;
      const int car0 = is_tail ? Lr - (it * G::KEYS_IT + tile * KT) : KT;  // carried keys: [car0, car0 + c)
      if (is_tail) softmax_store<true>(sc, sl2, neg, prow, r, car0, c, psum, pcar);
      else softmax_store<false>(sc, sl2, neg, prow, r, car0, c, psum, pcar);
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(smem_u32(p_full + (it & 1)));
      l_run += psum;
      lc_run += pcar;
    }

    // partial result of this row: O from tensor memory once the last PV has landed. With two
    // interleaved tiles, lanes l and l + 16 hold the same query row for different keys: they are
    // merged with shuffles (log-sum-exp weights) so the CTA writes one partial per row.
    if (ok && n_it > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(o_full + ((n_it - 1) & 1)), ((n_it - 1) >> 1) & 1, abort_flag, p.status));
      if (ok) {
        tc_fence_after();
        float w_me = 1.f, w_other = 0.f;
        float m_out = m_ref;
        if (DUAL) {
          const float m_o = __shfl_xor_sync(0xffffffffu, m_ref, 16);
          const float l_o = __shfl_xor_sync(0xffffffffu, l_run, 16), lc_o = __shfl_xor_sync(0xffffffffu, lc_run, 16);
          m_out = fmaxf(m_ref, m_o);
          const float base_m = m_out == -INFINITY ? 0.f : m_out;
          w_me = ex2_approx((m_ref - base_m) * sl2);
          w_other = ex2_approx((m_o - base_m) * sl2);
          l_run = w_me * l_run + w_other * l_o;
          lc_run = w_me * lc_run + w_other * lc_o;
        }
        const size_t rowi = ((static_cast<size_t>(s) * p.n_kv + h) * p.max_parts + split) * M + min(r, M - 1);
        float4* po = reinterpret_cast<float4*>(p.part_o + rowi * HD);
      const uint64_t pol_keep = l2_policy_evict_last();
#pragma unroll
        for (int q4 = 0; q4 < HD / 32; ++q4) {
          uint32_t v[32];
          tmem_ld32(t_lane + G::COL_O + q4 * 32, v);
          float o[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            o[j] = __uint_as_float(v[j]) * w_me;
            if (DUAL) o[j] += __shfl_xor_sync(0xffffffffu, __uint_as_float(v[j]), 16) * w_other;
          }
          // the two lanes of a row share the stores: even chunks from the first tile's lane
          if (r < M && (!DUAL || ((q4 & 1) == tile))) {
#pragma unroll
            for (int j = 0; j < 8; ++j) st_float4_hint(po + q4 * 8 + j, o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3], pol_keep);
          }
        }
        if (r < M && tile == 0) {
          float* ml = p.part_ml + rowi * 4;
          ml[0] = m_out * rsqrtf(static_cast<float>(HD));      // natural-log units of the scaled score
          ml[1] = l_run;
          ml[2] = lc_run;
        }
      }
    }
  }

  // ---------------------------------------------------- teardown
  if (flags) atomicOr(p.status, flags);
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, G::TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------------------
// The same attention as k_attn_tc for grids several waves deep, as a PERSISTENT kernel: two CTAs per SM walk the
// longest-first work list with a fixed stride, and the pipeline never drains between work items. All ring slots,
// score buffers and barrier phases are indexed by ONE step counter g that runs across items, so at an item
// boundary the producers simply keep going: the next item's first K/V tiles are requested as soon as the slots
// free up (the K producer also requests the next item's Q tile then, by TMA), and they stream while the soft-max
// threads store the finished item's partial result. What a one-item CTA pays per item - launch, barrier set-up,
// tensor-memory allocation, a Q gather, a first load with nothing else in flight, the drain - is paid once per
// CTA here; with ~2.7 items per CTA at batch 32 that was a fifth of the kernel's time (bytes in flight dip
// whenever CTAs turn over, and an HBM-bound kernel is only as fast as its bytes in flight).
// Differences inside an item: Q arrives by two 5-D TMA boxes instead of a gather; the page of each tile comes
// straight from the block table, one step ahead, into a register; tail items (partial page + carried + block
// rows, gathered with plain loads by the soft-max threads) complete their slot with one elected arrival, so a
// barrier serves TMA-fed and gathered tiles alike; the first PV of an item waits until the soft-max threads have
// read the previous item's O out of tensor memory (o_free).
// Twelve warps in three warpgroups: 0-3 soft-max; 4 the K (and Q) producer, 5 the MMA issuer, 6 the V producer;
// 7-11 only hand their registers over. After the common set-up the warpgroups rebalance their register budgets
// (setmaxnreg): the soft-max rows' 64 scores stay in registers at 144 per thread, everyone else keeps 48.
// The increase WAITS, without any bound, until the CTA's own pool holds the registers: the budgets must fit what
// the CTA was launched with (PS_REGS_LAUNCH per thread; the host checks the compiled kernel before the first launch),
// and ptxas applies a raised budget only to code inside the branch that executes the instruction.
constexpr int NTHREADS_PS = 384, PS_REGS_LAUNCH = 80, PS_REGS_SOFTMAX = 144, PS_REGS_OTHER = 48;
static_assert(128 * PS_REGS_SOFTMAX + (NTHREADS_PS - 128) * PS_REGS_OTHER <= NTHREADS_PS * PS_REGS_LAUNCH, "setmaxnreg budgets exceed the CTA's pool");
template <bool DUAL>
__global__ void __launch_bounds__(NTHREADS_PS, 2)
k_attn_ps(const __grid_constant__ CUtensorMap map_pool, const __grid_constant__ CUtensorMap map_zero,
          const __grid_constant__ CUtensorMap map_q, const AttnParams p) {
  cod_pdl_prologue();
  using G = Geo<DUAL>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + G::OFF_CTL);
  uint64_t* k_full = bars;                  // [NK]
  uint64_t* k_empty = bars + 5;             // [NK]
  uint64_t* v_full = bars + 10;             // [NV]
  uint64_t* v_empty = bars + 15;            // [NV]
  uint64_t* s_full = bars + 20;             // [2]
  uint64_t* p_full = bars + 22;             // [2]
  uint64_t* o_full = bars + 24;             // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint64_t* q_full = bars + 27;             // the item's Q tile has landed
  uint64_t* o_free = bars + 28;             // the previous item's O has been read out of tensor memory

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int M = p.W * p.rep;
  uint32_t flags = 0;

  // One work item = (sequence, KV head, part). Every role decodes the same sequence of items for this CTA.
  struct Item { int s, h, split, F, Lr, c, n_tail, k_begin, k_end, n_it; bool is_tail; uint32_t bad; };
  // Work unit w = list entry w / n_kv, head w % n_kv. A CTA's first unit is its own index; every further one is
  // the next the whole grid has not taken yet (a device counter): over the longest-first list that is the
  // longest-processing-time rule, which a fixed assignment cannot match when CTAs progress at different rates.
  // The K producer's first lane takes the unit and publishes it to the other roles through a small ring.
  int* witem = reinterpret_cast<int*>(bars + 40);     // [8]
  uint64_t* item_bar = bars + 32;                     // [8] unit j of this CTA has been published
  auto take_unit = [&](int j) {                       // (K producer, lane 0)
    int w = j == 0 ? static_cast<int>(blockIdx.x) : static_cast<int>(gridDim.x) + atomicAdd(p.work_counter, 1);
    if (w / p.n_kv >= p.n_list || p.order[w / p.n_kv] < 0) w = -1;      // the list is packed: nothing further
    witem[j & 7] = w;
    mbar_arrive(smem_u32(item_bar + (j & 7)));
  };
  auto unit_of = [&](int j, bool& ok) -> int {        // every role; ok false: a wait ran out
    ok = mbar_wait(smem_u32(item_bar + (j & 7)), (j >> 3) & 1, abort_flag, p.status);
    return ok ? witem[j & 7] : -1;
  };
  auto decode = [&](int w, Item& t) {
    const int idx = w / p.n_kv;
    const int item = p.order[idx];
    t.h = w - idx * p.n_kv; t.s = item >> 16; t.split = item & 0xFFFF;
    int L = p.committed_len[t.s];
    int c = p.use_carry ? p.carry_len[t.s] : 0;
    t.bad = 0;
    if (L < 0 || L > p.max_pages * PAGE) { t.bad = COD_DEV_BAD_LEN; L = max(0, min(L, p.max_pages * PAGE)); }
    if (c < 0 || c > p.cap) { t.bad = COD_DEV_BAD_LEN; c = max(0, min(c, p.cap)); }
    t.c = c;
    t.F = (L / PAGE) * PAGE;
    const int n_reg = (t.F + p.split_len - 1) / p.split_len;
    t.is_tail = t.split >= n_reg;                     // (the list holds existing parts only: == n_reg)
    t.Lr = L - t.F;
    t.n_tail = t.Lr + c + p.W;
    t.k_begin = t.is_tail ? 0 : t.split * p.split_len;
    t.k_end = t.is_tail ? t.n_tail : min(t.F, t.k_begin + p.split_len);
    t.n_it = (t.k_end - t.k_begin + G::KEYS_IT - 1) / G::KEYS_IT;
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < G::NK; ++i) { mbar_init(smem_u32(k_full + i), 1); mbar_init(smem_u32(k_empty + i), 1); }
    for (int i = 0; i < G::NV; ++i) { mbar_init(smem_u32(v_full + i), 1); mbar_init(smem_u32(v_empty + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(s_full + i), 1); mbar_init(smem_u32(p_full + i), 128); mbar_init(smem_u32(o_full + i), 1); }
    mbar_init(smem_u32(q_full), 1);
    mbar_init(smem_u32(o_free), 128);
    for (int i = 0; i < 8; ++i) mbar_init(smem_u32(item_bar + i), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(smem_u32(tmem_slot), G::TMEM_COLS);
  if (warp < 4) {
    // query rows beyond the real ones stay zero for the whole kernel (the Q boxes never touch them)
    for (int idx = threadIdx.x; idx < (G::MROWS - M) * 16; idx += 128) {
      const int r = M + (idx >> 4), ch = idx & 15;
      *reinterpret_cast<uint4*>(sm + (ch >> 3) * G::Q_HALF + r * 128 + ((ch & 7) << 4)) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp >= 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PS_REGS_OTHER));
  if (warp == 4 || warp == 6) {
    // ------------------------------------------------ TMA producers: warp 4 K tiles (and the Q tile), warp 6 V tiles
    const bool is_v = warp == 6;
    const int pages_it = G::KEYS_IT / PAGE;             // 8 or 4 pages per step, one per lane
    const int ring = is_v ? G::NV : G::NK;
    uint64_t* full = is_v ? v_full : k_full;
    uint64_t* empty = is_v ? v_empty : k_empty;
    const uint32_t ring_off = is_v ? G::OFF_V : G::OFF_K;
    const bool lane_on = lane < pages_it;
    const uint64_t pol_stream = l2_policy_evict_first();
    const uint32_t in_slot = (lane / (KT / PAGE)) * TILE_BYTES + (lane % (KT / PAGE)) * (PAGE * 128);
    int g = 0, j = 0;
    bool ok = true;
    Item t;
    for (;; ++j) {
      if (!is_v && lane == 0) take_unit(j);
      const int w = unit_of(j, ok);
      if (!ok || w < 0) break;
      decode(w, t);
      if (!is_v) {
        // Q of this item, once every QK of the previous item has retired (QKs retire in order)
        if (lane == 0 && g > 0) ok = mbar_wait(smem_u32(k_empty + (g - 1) % G::NK), ((g - 1) / G::NK) & 1, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane == 0) {
          const uint32_t qb = smem_u32(q_full);
          mbar_expect_tx(qb, static_cast<uint32_t>(M) * HD * 2);
          tma_load_5d(base, &map_q, 0, 0, 0, t.h, t.s * p.W, qb);
          tma_load_5d(base + G::Q_HALF, &map_q, 0, 1, 0, t.h, t.s * p.W, qb);
        }
      }
      if (!t.is_tail) {
        // this lane's physical page comes from the block table, one step ahead of its use
        const int* table = p.block_table + t.s * p.max_pages + t.k_begin / PAGE + lane;
        int pg_next = (lane_on && t.k_begin + lane * PAGE < t.k_end) ? table[0] : -1;
        for (int it = 0; it < t.n_it; ++it) {
          const int gg = g + it;
          const int key0 = t.k_begin + it * G::KEYS_IT + lane * PAGE;
          int pg = pg_next;
          if (lane_on && key0 + G::KEYS_IT < t.k_end) pg_next = table[(it + 1) * pages_it];
          int row = -1;                                 // first row of this lane's page tile in the pool map
          if (lane_on && key0 < t.k_end) {
            if (pg < 0 || pg >= p.n_pages) { flags |= COD_DEV_BAD_PAGE; pg = -1; }
            if (pg >= 0) row = (((p.layer * p.n_pages + pg) * p.n_kv + t.h) * 2 + (is_v ? 1 : 0)) * PAGE;
          }
          const int slot = gg % ring, use = gg / ring;
          if (lane == 0 && use > 0) ok = mbar_wait(smem_u32(empty + slot), (use - 1) & 1, abort_flag, p.status);
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
          const uint32_t fb = smem_u32(full + slot);
          if (lane == 0) mbar_expect_tx(fb, G::SLOT);
          __syncwarp();
          if (lane_on) {
            const uint32_t dst = base + ring_off + slot * G::SLOT + in_slot;
            if (row >= 0) {
              tma_load_3d_hint(dst, &map_pool, 0, 0, row, fb, pol_stream);
              tma_load_3d_hint(dst + HALF_BYTES, &map_pool, 0, 1, row, fb, pol_stream);
            } else {
              tma_load_3d(dst, &map_zero, 0, 0, 0, fb);
              tma_load_3d(dst + HALF_BYTES, &map_zero, 0, 1, 0, fb);
            }
          }
        }
      }
      if (!ok) break;
      g += t.n_it;
    }
  } else if (warp == 5) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc(G::MROWS, KT, 0);
      const uint32_t idesc_pv = instr_desc(G::MROWS, HD, 1);
      const uint64_t q_desc = desc_kmajor_sw128(base);
      bool ok = true;
      auto issue_qk = [&](int gg) -> bool {
        const int slot = gg % G::NK;
        if (!mbar_wait(smem_u32(k_full + slot), (gg / G::NK) & 1, abort_flag, p.status)) return false;
        tc_fence_after();
#pragma unroll
        for (int tl = 0; tl < G::TILES; ++tl) {
          const uint64_t k_desc = desc_kmajor_sw128(base + G::OFF_K + slot * G::SLOT + tl * TILE_BYTES);
          const uint32_t d = tmem_base + G::COL_S + (gg & 1) * KT + (static_cast<uint32_t>(16 * tl) << 16);
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            const uint32_t qa = (k < 4 ? 0u : (G::Q_HALF >> 4)) + (k & 3) * 2;
            const uint32_t ka = (k < 4 ? 0u : (HALF_BYTES >> 4)) + (k & 3) * 2;
            umma_bf16(d, q_desc + qa, k_desc + ka, idesc_qk, k ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(s_full + (gg & 1)));
        umma_commit(smem_u32(k_empty + slot));
        return true;
      };
      int g = 0, j = 0;
      Item t;
      for (;; ++j) {
        const int w = unit_of(j, ok);
        if (!ok || w < 0) break;
        decode(w, t);
        ok = mbar_wait(smem_u32(q_full), j & 1, abort_flag, p.status);
        if (!ok) break;
        ok = issue_qk(g);
        for (int it = 0; it < t.n_it && ok; ++it) {
          const int gg = g + it;
          if (it + 1 < t.n_it) ok = issue_qk(gg + 1);
          if (!ok) break;
          const int slot = gg % G::NV;
          ok = mbar_wait(smem_u32(p_full + (gg & 1)), (gg >> 1) & 1, abort_flag, p.status) &&
               mbar_wait(smem_u32(v_full + slot), (gg / G::NV) & 1, abort_flag, p.status);
          // the first PV of an item overwrites O: the previous item's O must have been read
          if (ok && it == 0 && j > 0) ok = mbar_wait(smem_u32(o_free), (j - 1) & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int tl = 0; tl < G::TILES; ++tl) {
            const uint64_t p_desc = desc_kmajor_sw128(base + G::OFF_P + tl * G::P_TILE);
            const uint64_t v_desc = desc_mnmajor_sw128(base + G::OFF_V + slot * G::SLOT + tl * TILE_BYTES, HALF_BYTES);
            const uint32_t d = tmem_base + G::COL_O + (static_cast<uint32_t>(16 * tl) << 16);
#pragma unroll
            for (int kk = 0; kk < KT / 16; ++kk)       // 16 keys per MMA: 32 bytes along P's rows, 16 rows of V
              umma_bf16(d, p_desc + kk * 2, v_desc + kk * ((16 * 128) >> 4), idesc_pv, (it | kk) ? 1u : 0u);
          }
          umma_commit(smem_u32(o_full + (gg & 1)));
          umma_commit(smem_u32(v_empty + slot));
        }
        if (!ok) break;
        g += t.n_it;
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(PS_REGS_SOFTMAX));
    // ------------------------------------------------ softmax: one thread per (row, tile), as in k_attn_tc
    const int T = threadIdx.x;
    const int tile = DUAL ? (lane >> 4) : 0;
    const int r = DUAL ? (16 * warp + (lane & 15)) : T;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(32 * warp) << 16);
    const float sl2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;   // raw score -> log2 units
    const float rescale_gap = 8.f / sl2;
    bool ok = true;
    int g = 0, j = 0;
    Item t;
    for (;; ++j) {
      const int w = unit_of(j, ok);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok || w < 0) break;
      decode(w, t);
      float m_ref = -INFINITY, l_run = 0.f, lc_run = 0.f;
      const int s = t.s, h = t.h, c = t.c, Lr = t.Lr, F = t.F, n_it = t.n_it, k_begin = t.k_begin, k_end = t.k_end,
                n_tail = t.n_tail, split = t.split;
      const bool is_tail = t.is_tail;
      flags |= t.bad;
#pragma unroll 1
      for (int it = 0; it < n_it && ok; ++it) {
        const int gg = g + it;
        if (is_tail) {
          // gather this step's rows (partial page, carried rows, block rows) with plain loads: first the K
          // rows (the MMA warp asks for them first), then the V rows; one elected arrival completes the slot
          constexpr int GB = 8;                               // independent 16-byte loads in flight per thread
#pragma unroll 1
          for (int kv = 0; kv < 2; ++kv) {
            const int ring = kv ? G::NV : G::NK;
            const int slot = gg % ring, use = gg / ring;
            uint64_t* full = kv ? v_full : k_full;
            uint64_t* empty = kv ? v_empty : k_empty;
            if (use > 0) {
              ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(empty + slot), (use - 1) & 1, abort_flag, p.status));
              if (!ok) break;
            }
            for (int idx0 = T; idx0 < G::KEYS_IT * 16; idx0 += 128 * GB) {
              uint4 val[GB];
              uint32_t dst[GB];
#pragma unroll
              for (int u = 0; u < GB; ++u) {
                const int idx = idx0 + u * 128;
                const int ch = idx & 15, jk = idx >> 4;                         // chunk, key within the step
                const int gk = it * G::KEYS_IT + jk;
                const __nv_bfloat16* src = nullptr;
                if (gk < Lr) {
                  int pg = p.block_table[s * p.max_pages + F / PAGE];
                  if (pg < 0 || pg >= p.n_pages) { flags |= COD_DEV_BAD_PAGE; }
                  else src = p.pool + ((((static_cast<size_t>(p.layer) * p.n_pages + pg) * p.n_kv + h) * 2 + kv) * PAGE + gk) * HD;
                } else if (gk < Lr + c) {
                  src = p.carry + ((((static_cast<size_t>(p.layer) * p.max_batch + s) * p.n_kv + h) * 2 + kv) * p.cap + (gk - Lr)) * HD;
                } else if (gk < n_tail) {
                  src = (kv ? p.vb : p.kb) + static_cast<size_t>(s * p.W + (gk - Lr - c)) * (p.n_kv * HD) + h * HD;
                }
                val[u] = src ? *reinterpret_cast<const uint4*>(src + ch * 8) : make_uint4(0u, 0u, 0u, 0u);
                const int jj = jk & (KT - 1), tl = jk / KT;
                dst[u] = (kv ? G::OFF_V : G::OFF_K) + slot * G::SLOT + tl * TILE_BYTES +
                         (ch >> 3) * HALF_BYTES + jj * 128 + (((ch & 7) ^ (jj & 7)) << 4);
              }
#pragma unroll
              for (int u = 0; u < GB; ++u) *reinterpret_cast<uint4*>(sm + dst[u]) = val[u];
            }
            fence_async_smem();
            asm volatile("bar.sync 2, 128;" ::: "memory");
            if (T == 0) mbar_arrive(smem_u32(full + slot));
          }
          if (!ok) break;
        }

        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(s_full + (gg & 1)), (gg >> 1) & 1, abort_flag, p.status));
        if (!ok) break;
        tc_fence_after();
        const int key_t0 = k_begin + it * G::KEYS_IT + tile * KT;         // first key of this thread's tile
        const int n_valid = max(0, min(KT, k_end - key_t0));
        float sc[KT];
        {
          uint32_t v[32];
          tmem_ld32(t_lane + G::COL_S + (gg & 1) * KT, v);
#pragma unroll
          for (int q = 0; q < 32; ++q) sc[q] = __uint_as_float(v[q]);
          tmem_ld32(t_lane + G::COL_S + (gg & 1) * KT + 32, v);
#pragma unroll
          for (int q = 0; q < 32; ++q) sc[32 + q] = __uint_as_float(v[q]);
        }
        if (n_valid < KT) {                                  // only the last step of a part is ragged
#pragma unroll
          for (int q = 0; q < KT; ++q) sc[q] = q < n_valid ? sc[q] : -INFINITY;
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};      // four independent chains
#pragma unroll
        for (int q = 0; q < KT; q += 4) {
          mx4[0] = fmaxf(mx4[0], sc[q]); mx4[1] = fmaxf(mx4[1], sc[q + 1]);
          mx4[2] = fmaxf(mx4[2], sc[q + 2]); mx4[3] = fmaxf(mx4[3], sc[q + 3]);
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const bool need = mx > m_ref + rescale_gap;        // also true for the first finite maximum
        if (__any_sync(0xffffffffu, need)) {
          const float m_new = need ? mx : m_ref;
          const float factor = need ? ex2_approx((m_ref - m_new) * sl2) : 1.f;     // ex2(-inf) = 0
          if (it > 0) {
            // O is relative to the old reference: once PV(g-1) has landed, scale this warp's rows
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(o_full + ((gg - 1) & 1)), ((gg - 1) >> 1) & 1, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int q4 = 0; q4 < HD / 32; ++q4) {
              uint32_t v[32];
              tmem_ld32(t_lane + G::COL_O + q4 * 32, v);
#pragma unroll
              for (int q = 0; q < 32; ++q) v[q] = __float_as_uint(__uint_as_float(v[q]) * factor);
              tmem_st32(t_lane + G::COL_O + q4 * 32, v);
            }
          }
          l_run *= factor;
          lc_run *= factor;
          m_ref = m_new;
        }
        if (gg >= 1) {   // the P buffer about to be overwritten was read by PV(g-1) (possibly the previous item's last)
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(o_full + ((gg - 1) & 1)), ((gg - 1) >> 1) & 1, abort_flag, p.status));
          if (!ok) break;
        }
        const float neg = m_ref == -INFINITY ? 0.f : -m_ref * sl2;
        float psum, pcar;
        uint8_t* prow = sm + G::OFF_P + tile * G::P_TILE + r * 128;
        const int car0 = is_tail ? Lr - (it * G::KEYS_IT + tile * KT) : KT;  // carried keys: [car0, car0 + c)
        if (is_tail) softmax_store<true>(sc, sl2, neg, prow, r, car0, c, psum, pcar);
        else softmax_store<false>(sc, sl2, neg, prow, r, car0, c, psum, pcar);
        fence_async_smem();
        tc_fence_before();
        mbar_arrive(smem_u32(p_full + (gg & 1)));
        l_run += psum;
        lc_run += pcar;
      }
      if (!ok) break;

      // the item's partial result: O out of tensor memory once its last PV has landed (see k_attn_tc), then
      // the accumulator is handed back to the MMA issuer
      const int gl = g + n_it - 1;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(o_full + (gl & 1)), (gl >> 1) & 1, abort_flag, p.status));
      if (!ok) break;
      tc_fence_after();
      float w_me = 1.f, w_other = 0.f;
      float m_out = m_ref;
      if (DUAL) {
        const float m_o = __shfl_xor_sync(0xffffffffu, m_ref, 16);
        const float l_o = __shfl_xor_sync(0xffffffffu, l_run, 16), lc_o = __shfl_xor_sync(0xffffffffu, lc_run, 16);
        m_out = fmaxf(m_ref, m_o);
        const float base_m = m_out == -INFINITY ? 0.f : m_out;
        w_me = ex2_approx((m_ref - base_m) * sl2);
        w_other = ex2_approx((m_o - base_m) * sl2);
        l_run = w_me * l_run + w_other * l_o;
        lc_run = w_me * lc_run + w_other * lc_o;
      }
      const size_t rowi = ((static_cast<size_t>(s) * p.n_kv + h) * p.max_parts + split) * M + min(r, M - 1);
      float4* po = reinterpret_cast<float4*>(p.part_o + rowi * HD);
      const uint64_t pol_keep = l2_policy_evict_last();
#pragma unroll
      for (int q4 = 0; q4 < HD / 32; ++q4) {
        uint32_t v[32];
        tmem_ld32(t_lane + G::COL_O + q4 * 32, v);
        float o[32];
#pragma unroll
        for (int q = 0; q < 32; ++q) {
          o[q] = __uint_as_float(v[q]) * w_me;
          if (DUAL) o[q] += __shfl_xor_sync(0xffffffffu, __uint_as_float(v[q]), 16) * w_other;
        }
        if (q4 == HD / 32 - 1) {                            // every column has been read: O may be overwritten
          tc_fence_before();
          mbar_arrive(smem_u32(o_free));
        }
        // the two lanes of a row share the stores: even chunks from the first tile's lane
        if (r < M && (!DUAL || ((q4 & 1) == tile))) {
#pragma unroll
          for (int q = 0; q < 8; ++q) st_float4_hint(po + q4 * 8 + q, o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3], pol_keep);
        }
      }
      if (r < M && tile == 0) {
        float* ml = p.part_ml + rowi * 4;
        ml[0] = m_out * rsqrtf(static_cast<float>(HD));      // natural-log units of the scaled score
        ml[1] = l_run;
        ml[2] = lc_run;
      }
      g += n_it;
    }
  }

  // ---------------------------------------------------- teardown
  if (flags) atomicOr(p.status, flags);
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, G::TMEM_COLS);
  }
}

// Work order for grids several waves deep: every (sequence, part) that exists, longest first, so the
// last wave is made of short parts instead of whichever sequences come last (a counting sort by
// iteration count in one block; the order inside a bucket is arbitrary and affects no result).
template <int KEYS_IT>
__global__ void k_attn_order(const int* __restrict__ committed_len, int S, int max_pages, int split_len,
                             int max_parts, int* __restrict__ order) {
  cod_pdl_prologue();
  constexpr int NB = 4096 / 64 + 3;              // keys: 0 absent, 1 tail, 1 + iterations of a paged part
  __shared__ int hist[NB], cur[NB], n_items;
  for (int k = threadIdx.x; k < NB; k += blockDim.x) hist[k] = 0;
  __syncthreads();
  const int n_max = S * max_parts;
  auto key_of = [&](int i) -> int {
    const int s = i / max_parts, split = i - s * max_parts;
    const int L = max(0, min(committed_len[s], max_pages * PAGE));
    const int F = (L / PAGE) * PAGE;
    const int n_reg = (F + split_len - 1) / split_len;
    if (split > n_reg) return 0;
    if (split == n_reg) return 1;
    const int keys = min(F, (split + 1) * split_len) - split * split_len;
    return min(NB - 1, 1 + (keys + KEYS_IT - 1) / KEYS_IT);
  };
  for (int i = threadIdx.x; i < n_max; i += blockDim.x) atomicAdd(&hist[key_of(i)], 1);
  __syncthreads();
  if (threadIdx.x == 0) {
    int pos = 0;
    for (int k = NB - 1; k >= 1; --k) { cur[k] = pos; pos += hist[k]; }
    n_items = pos;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n_max; i += blockDim.x) {
    const int k = key_of(i);
    if (k > 0) {
      const int s = i / max_parts;
      order[atomicAdd(&cur[k], 1)] = (s << 16) | (i - s * max_parts);
    }
  }
  for (int i = n_items + threadIdx.x; i < n_max; i += blockDim.x) order[i] = -1;
}

// Merges the partials of one (row, query head); one warp each. Empty partials carry m = -inf, l = 0.
// FEW: no (sequence, head) has more than four parts (large batches: long parts). The kernel is bound by how many
// warps wait on L2 at once, and without the eight-row batches of the general loop it fits eight blocks per SM.
template <bool DUAL, bool FEW>
__global__ void __launch_bounds__(128, FEW ? 8 : 1) k_attn_tc_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                                  const int* __restrict__ committed_len, int S, int W, int rep, int n_kv,
                                  int max_pages, int split_len, int max_parts, __nv_bfloat16* __restrict__ out,
                                  float* __restrict__ tap, float* __restrict__ mass, int* __restrict__ work_counter, int drop) {
  cod_pdl_prologue();
  if (work_counter != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *work_counter = 0;   // for the next persistent attention launch
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int n_q = n_kv * rep;
  if (item >= S * W * n_q) return;
  const int g = item % n_q, i = (item / n_q) % W, s = item / (n_q * W);
  const int h = g / rep, mrow = i * rep + (g - h * rep), M = W * rep;
  const int L = max(0, min(committed_len[s], max_pages * PAGE));
  const int F = (L / PAGE) * PAGE;
  const int n_parts = (F + split_len - 1) / split_len + 1;
  const size_t base = (static_cast<size_t>(s) * n_kv + h) * max_parts;
  // The first four partial rows are requested together with the (m, l, l_carry) records (they need only
  // the part count): at large batches the partials have left L2 by now and every dependent trip costs.
  // Every lane fetches the record of its parts once; weights stay in registers.
  constexpr int C0 = 4;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 v0[C0];
#pragma unroll
  for (int u = 0; u < C0; ++u)
    v0[u] = u < n_parts ? *reinterpret_cast<const float4*>(part_o + ((base + u) * M + mrow) * HD + lane * 4) : zero4;
  const float4 none = make_float4(-INFINITY, 0.f, 0.f, 0.f);
  const float4 ml0 = lane < n_parts ? *reinterpret_cast<const float4*>(part_ml + ((base + lane) * M + mrow) * 4) : none;
  float mg = ml0.x;
  for (int k = lane + 32; k < n_parts; k += 32) mg = fmaxf(mg, part_ml[((base + k) * M + mrow) * 4]);
  mg = cod_warp_max(mg);
  float acc[4] = {0.f, 0.f, 0.f, 0.f}, l = 0.f, lc = 0.f;
  for (int k0 = 0; k0 < n_parts; k0 += 32) {
    float4 ml = ml0;
    if (k0 > 0) ml = k0 + lane < n_parts ? *reinterpret_cast<const float4*>(part_ml + ((base + k0 + lane) * M + mrow) * 4) : none;
    const float w_mine = k0 + lane < n_parts ? __expf(ml.x - mg) : 0.f;
    l = fmaf(w_mine, ml.y, l);
    lc = fmaf(w_mine, ml.z, lc);
    const int nk = min(32, n_parts - k0);
    int kk = 0;
    if (k0 == 0) {
#pragma unroll
      for (int u = 0; u < C0; ++u) {
        const float w = __shfl_sync(0xffffffffu, w_mine, u);                  // lanes past the last part hold 0
        acc[0] = fmaf(w, v0[u].x, acc[0]); acc[1] = fmaf(w, v0[u].y, acc[1]); acc[2] = fmaf(w, v0[u].z, acc[2]); acc[3] = fmaf(w, v0[u].w, acc[3]);
      }
      kk = C0;
    }
    // then eight partial rows at a time, their loads all in flight before the first is used (a batch-1
    // round merges 17 partials per head)
    if (!FEW)
    for (; kk < nk; kk += 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        v[u] = kk + u < nk ? *reinterpret_cast<const float4*>(part_o + ((base + k0 + kk + u) * M + mrow) * HD + lane * 4) : zero4;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float w = __shfl_sync(0xffffffffu, w_mine, (kk + u) & 31);
        acc[0] = fmaf(w, v[u].x, acc[0]); acc[1] = fmaf(w, v[u].y, acc[1]); acc[2] = fmaf(w, v[u].z, acc[2]); acc[3] = fmaf(w, v[u].w, acc[3]);
      }
    }
  }
  l = cod_warp_sum(l);
  lc = cod_warp_sum(lc);
  // this warp was the only reader of its partial rows (512 bytes each): they are dead now and leave L2 without a
  // write-back (the warp barrier orders every lane's reads before the drop)
  __syncwarp();
  if (drop)
    for (int k = lane & 7; k < n_parts; k += 8)         // a lane drops the line its own 16 bytes came from, for every eighth part
      cod_discard_line(part_o + ((base + k) * M + mrow) * HD + (lane >> 3) * 32);
  const float inv = 1.f / l;
  const size_t ob = static_cast<size_t>(item) * HD + lane * 4;
  const __nv_bfloat162 b0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv), b1 = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
  uint2 pk;
  pk.x = *reinterpret_cast<const uint32_t*>(&b0);
  pk.y = *reinterpret_cast<const uint32_t*>(&b1);
  *reinterpret_cast<uint2*>(out + ob) = pk;
  if (tap) *reinterpret_cast<float4*>(tap + ob) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
  if (mass && lane == 0) mass[item] = lc * inv;
}


template <bool DUAL>
int launch(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb, const cod_state* stt, int S,
           int use_carry, void* out, float* tap, float* mass, cudaStream_t st) {
  using G = Geo<DUAL>;
  const cod_config& f = c->cfg;
  CUtensorMap mp, mz;
  const uint64_t rows = static_cast<uint64_t>(f.n_layers) * f.n_pages * f.n_kv_heads * 2 * PAGE;
  if (!make_map_rows128(&mp, stt->kv_pool, rows, PAGE) || !make_map_rows128(&mz, c->zero_page, PAGE, PAGE)) return COD_ERR_CUDA;
  AttnParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q); p.kb = static_cast<const __nv_bfloat16*>(kb); p.vb = static_cast<const __nv_bfloat16*>(vb);
  p.pool = static_cast<const __nv_bfloat16*>(stt->kv_pool); p.carry = static_cast<const __nv_bfloat16*>(stt->carry_kv);
  p.block_table = stt->block_table; p.committed_len = stt->committed_len; p.carry_len = stt->carry_len;
  p.cap = c->carry_cap;
  p.use_carry = use_carry; p.layer = layer; p.W = f.block; p.rep = f.n_q_heads / f.n_kv_heads; p.n_kv = f.n_kv_heads;
  p.n_pages = f.n_pages; p.max_pages = f.max_pages_per_seq; p.max_batch = f.max_batch;
  p.split_len = c->tc_split_len; p.max_parts = c->tc_max_parts;
  p.part_o = c->attn_o; p.part_ml = c->attn_ml; p.status = c->status;
  p.run_ahead = c->attn_run_ahead ? 1 : 0;
  // the attribute belongs to (kernel, device): one flag per device the process may use
  static bool configured_dev[64] = {};
  bool& configured = configured_dev[c->device & 63];
  if (!configured) {
    if (cudaFuncSetAttribute(k_attn_tc<DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(G::SMEM)) != cudaSuccess)
      return COD_ERR_CUDA;
    configured = true;
  }
  dim3 grid(c->tc_max_parts, f.n_kv_heads, S);
  // more CTAs than fit on the machine at once: longest parts first (the list holds until the lengths change)
  if (c->attn_order != nullptr && static_cast<long long>(S) * f.n_kv_heads * c->tc_max_parts > 2ll * c->n_sm && S < 32768 &&
      static_cast<long long>(S) * c->tc_max_parts <= 65535) {
    if (c->attn_order_stale) {
      cod_launch_pdl(c, k_attn_order<G::KEYS_IT>, 1, 256, 0, st, stt->committed_len, S, f.max_pages_per_seq, c->tc_split_len,
                     c->tc_max_parts, c->attn_order);
      COD_CHECK_LAUNCH(c);
      c->attn_order_stale = false;
    }
    p.order = c->attn_order;
    p.n_list = S * c->tc_max_parts;
    p.work_counter = c->attn_counter;
    grid = dim3(f.n_kv_heads, S * c->tc_max_parts, 1);
    // the persistent form: two CTAs per SM walk the list (query rows must fill whole boxes: M = W * rep)
    CUtensorMap mq;
    // (measured: with 128 query rows per head group - block 32 - the persistent form is 7 % faster at 4 x 32K keys;
    // with 64 rows the two interleaved tiles already keep HBM at what it gives this access pattern, ~6 TB/s, and
    // the one-item CTAs of the hardware scheduler come out 6 % ahead at batch 32, so they stay)
    if ((!DUAL || c->attn_persistent) && !c->attn_one_item_ctas &&
        make_map_q(&mq, q, static_cast<uint64_t>(f.max_batch) * f.block, p.rep, f.n_kv_heads, f.block)) {
      static bool configured_ps[64] = {};
      if (!configured_ps[c->device & 63]) {
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, k_attn_ps<DUAL>) != cudaSuccess) return COD_ERR_CUDA;
        if (fa.numRegs < PS_REGS_LAUNCH) return COD_ERR_UNSUPPORTED;   // the CTA's register pool would be smaller than the budgets assume
        if (cudaFuncSetAttribute(k_attn_ps<DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(G::SMEM)) != cudaSuccess)
          return COD_ERR_CUDA;
        configured_ps[c->device & 63] = true;
      }
      const long long work = static_cast<long long>(S) * c->tc_max_parts * f.n_kv_heads;
      const int groups = 2 * c->n_sm / f.n_kv_heads > 0 ? 2 * c->n_sm / f.n_kv_heads : 1;          // head groups resident at once
      const int ctas = static_cast<int>(work / f.n_kv_heads < groups ? work : static_cast<long long>(groups) * f.n_kv_heads);
      cod_launch_pdl(c, k_attn_ps<DUAL>, dim3(ctas, 1, 1), NTHREADS_PS, G::SMEM, st, mp, mz, mq, p);
      COD_CHECK_LAUNCH(c);
    } else {
      cod_launch_pdl(c, k_attn_tc<DUAL>, grid, NTHREADS, G::SMEM, st, mp, mz, p);
      COD_CHECK_LAUNCH(c);
    }
  } else {
    cod_launch_pdl(c, k_attn_tc<DUAL>, grid, NTHREADS, G::SMEM, st, mp, mz, p);
    COD_CHECK_LAUNCH(c);
  }
  const int items = S * f.block * f.n_q_heads;
  // partials worth dropping from L2 once merged: when the launch may have written more than a few MB of them
  const int drop = static_cast<long long>(S) * f.n_kv_heads * c->tc_max_parts * f.block * p.rep * HD * 4 > (8ll << 20) ? 1 : 0;
  if (c->tc_max_parts <= 4)
    cod_launch_pdl(c, k_attn_tc_combine<DUAL, true>, (items + 3) / 4, 128, 0, st, c->attn_o, c->attn_ml, stt->committed_len, S, f.block, p.rep,
                   f.n_kv_heads, f.max_pages_per_seq, c->tc_split_len, c->tc_max_parts, static_cast<__nv_bfloat16*>(out), tap, mass,
                   c->attn_counter, drop);
  else
    cod_launch_pdl(c, k_attn_tc_combine<DUAL, false>, (items + 3) / 4, 128, 0, st, c->attn_o, c->attn_ml, stt->committed_len, S, f.block, p.rep,
                   f.n_kv_heads, f.max_pages_per_seq, c->tc_split_len, c->tc_max_parts, static_cast<__nv_bfloat16*>(out), tap, mass,
                   c->attn_counter, drop);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

}  // namespace

bool cod_attn_tc_supported(const cod_ctx* c) {
  const cod_config& f = c->cfg;
  const int M = f.block * (f.n_q_heads / f.n_kv_heads);
  return f.dtype == COD_BF16 && f.head_dim == HD && f.page_size == PAGE && M <= 128 && !c->force_simt &&
         c->tc_max_parts > 0 && encode_fn() != nullptr;
}

// q / kb already rotated. Layout of the partial buffers is private to this file.
int cod_launch_attn_tc(cod_ctx* c, int layer, const void* q, const void* kb, const void* vb, const cod_state* stt,
                       int S, int use_carry, void* out, float* tap, float* mass, cudaStream_t st) {
  const int M = c->cfg.block * (c->cfg.n_q_heads / c->cfg.n_kv_heads);
  if (M <= 64) return launch<true>(c, layer, q, kb, vb, stt, S, use_carry, out, tap, mass, st);
  return launch<false>(c, layer, q, kb, vb, stt, S, use_carry, out, tap, mass, st);
}
