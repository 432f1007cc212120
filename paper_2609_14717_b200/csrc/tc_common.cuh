// PTX wrappers and descriptor builders shared by the tensor-core kernels (tcgen05 + TMA, sm_100a).
// Everything here is a thin, named layer over one instruction or one bit layout.
#pragma once

#include <cuda.h>

#include "cod_internal.cuh"

namespace tc {

constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about 2 s at the maximum SM clock
constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;             // shared::cluster address -> the even-ranked CTA's copy

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// ---------------------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait. The common case (phase already complete, or completing within a few polls) never
// reads a timer; after that the SM cycle counter bounds the wait, then the CTA raises
// COD_DEV_TIMEOUT and every role leaves through the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* status,
                                          long long limit = WAIT_LIMIT_CYCLES) {
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      atomicOr(status, COD_DEV_TIMEOUT);
      return false;
    }
  }
}

// ---------------------------------------------------------------------------- TMA (one destination CTA each)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar) : "memory");
}
// untiled bulk copy of `bytes` contiguous bytes (both addresses 16-byte aligned, bytes a multiple of 16)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}
// paired-CTA form: the copy lands in THIS CTA's shared memory, its bytes are counted on the leader's barrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t leader_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(leader_bar) : "memory");
}

// ---------------------------------------------------------------------------- fences, cluster barrier
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
        "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
        "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------- MMA
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 operands, float accumulator; issued by one thread
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier is arrived on once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// paired form: M spans the tensor memory of both CTAs, each CTA supplies half of the B rows
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  const uint32_t z = 0u;   // no accumulator lane is masked off
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z) : "memory");
}
// arrive on the barrier at this offset in every CTA of the mask once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(cta_mask) : "memory");
}

// ---------------------------------------------------------------------------- descriptors
// Shared-memory operand, K-major: rows of 128 bytes (64 bf16), 128-byte swizzle, groups of 8 rows
// 1024 bytes apart; descriptor version 1 (Blackwell). Advancing 16 elements along K = +2 (32 bytes >> 4).
__device__ __forceinline__ uint64_t desc_kmajor_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);          // start address            bits [0,14)
  d |= static_cast<uint64_t>(1) << 16;                          // leading byte offset (unused for swizzled K-major)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                  // stride byte offset        bits [32,46)
  d |= static_cast<uint64_t>(1) << 46;                          // version                   bits [46,48)
  d |= static_cast<uint64_t>(2) << 61;                          // layout: 128-byte swizzle  bits [61,64)
  return d;
}
// MN-major operand (rows are K indices, 64 contiguous MN elements per 128-byte row): the next 64 MN
// elements sit lead_bytes further, the next 8 K indices 1024 bytes further.
__device__ __forceinline__ uint64_t desc_mnmajor_sw128(uint32_t saddr, uint32_t lead_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(lead_bytes >> 4) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// Instruction descriptor: bf16 x bf16 -> float, A K-major, B K-major or MN-major, shape m x n (x 16)
__device__ __forceinline__ uint32_t instr_desc(int m, int n, int b_mn_major) {
  uint32_t d = 0;
  d |= 1u << 4;                                  // accumulator format: float
  d |= 1u << 7;                                  // A format: bf16
  d |= 1u << 10;                                 // B format: bf16
  d |= static_cast<uint32_t>(b_mn_major) << 16;  // B major
  d |= static_cast<uint32_t>(n >> 3) << 17;      // N / 8
  d |= static_cast<uint32_t>(m >> 4) << 24;      // M / 16
  return d;
}

// ---------------------------------------------------------------------------- small arithmetic
__device__ __forceinline__ unsigned order_key(float v) {      // unsigned order = float order
  const unsigned u = __float_as_uint(v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Column-wise maximum over the 32 lanes of a warp for 32 columns at once: every lane brings one
// packed key per column; after five exchange rounds (16 + 8 + 4 + 2 + 1 shuffles) lane L holds
// the maximum of column L. The keys carry the row index, so this is an argmax with the lowest
// row winning ties.
__device__ __forceinline__ unsigned long long warp_colmax32(unsigned long long (&k)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool hi = (lane & off) != 0;
#pragma unroll
    for (int c = 0; c < off; ++c) {
      const unsigned long long send = hi ? k[c] : k[c + off];
      const unsigned long long mine = hi ? k[c + off] : k[c];
      const unsigned long long recv = __shfl_xor_sync(0xffffffffu, send, off);
      k[c] = recv > mine ? recv : mine;
    }
  }
  return k[0];
}

// Column-wise sum over the 32 lanes of a warp for 32 columns at once (same exchange pattern as
// warp_colmax32): afterwards lane L holds the sum of column L.
__device__ __forceinline__ float warp_colsum32(float (&e)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool hi = (lane & off) != 0;
#pragma unroll
    for (int c = 0; c < off; ++c) {
      const float send = hi ? e[c] : e[c + off];
      const float mine = hi ? e[c + off] : e[c];
      e[c] = mine + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return e[0];
}
__device__ __forceinline__ float order_key_to_float(unsigned k) {     // inverse of order_key
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// ---------------------------------------------------------------------------- sampling head
// Counter-based uniform number of the Gumbel-max draw: a chain of the 32-bit 'murmur3 finaliser'
// over (seed, step, row, column); U = ((h >> 9) + 0.5) * 2^-23 lies in (0, 1) and is exact in float.
__host__ __device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x85EBCA6Bu; x ^= x >> 13; x *= 0xC2B2AE35u; x ^= x >> 16;
  return x;
}
__host__ __device__ __forceinline__ uint32_t sample_state(unsigned long long seed, uint32_t step) {
  uint32_t h = mix32(static_cast<uint32_t>(seed) ^ 0x9E3779B9u);
  h = mix32(h + static_cast<uint32_t>(seed >> 32));
  return mix32(h + step);
}
// -log(-log U) for the element (row state h_row = mix32(state + row), column col). U comes within
// 2^-24 of 1, where -log U must keep its relative accuracy (those are the large-noise elements that
// tend to win the argmax): there -log U = -log1p(-w) with w = 1 - U (exact in float) is taken from
// its series, elsewhere from the fast logarithm; the outer logarithm's argument is never near 1 in
// relative terms that matter (absolute error 2^-22).
__device__ __forceinline__ float gumbel_noise(uint32_t h_row, uint32_t col) {
  const uint32_t h = mix32(h_row + col);
  const float u = (static_cast<float>(h >> 9) + 0.5f) * 1.1920928955078125e-07f;   // 2^-23
  const float w = 1.0f - u;
  const float t_series = w * fmaf(w, fmaf(w, 0.3333333433f, 0.5f), 1.0f);          // w < 2^-6: error < w^3 / 4
  const float t = w < 0.015625f ? t_series : -__logf(u);
  return -__logf(t);
}
// One chunk of 32 token columns in one warp of the LM-head epilogue, sampling form. v: the raw
// logits of this lane's vocabulary row (index vocab_idx, valid if f_ok) for the 32 columns;
// hrow: the 32 columns' row states. Returns for column `lane`: the packed (perturbed logit,
// ~index) key of the warp's best row, and the sum of exp(raw - m) over the warp's valid rows
// with m = that best perturbed logit (noise >= -2.9, so raw - m <= 2.9: no overflow).
__device__ __forceinline__ void sample_chunk(const uint32_t (&v)[32], bool f_ok, uint32_t vocab_idx,
                                             const uint32_t* hrow, int lane, unsigned long long& best,
                                             float& m_ref, float& s_sum) {
  const unsigned long long low = static_cast<unsigned long long>(0xFFFFFFFFu - vocab_idx);
  unsigned long long k[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const float pert = __uint_as_float(v[j]) + gumbel_noise(hrow[j], vocab_idx);
    k[j] = f_ok ? ((static_cast<unsigned long long>(order_key(pert)) << 32) | low) : 0ull;
  }
  best = warp_colmax32(k, lane);
  m_ref = best ? order_key_to_float(static_cast<unsigned>(best >> 32)) : -INFINITY;
  float e[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const float mj = __shfl_sync(0xffffffffu, m_ref, j);
    e[j] = (f_ok && mj > -INFINITY) ? __expf(__uint_as_float(v[j]) - mj) : 0.f;
  }
  s_sum = warp_colsum32(e, lane);
}

// ---------------------------------------------------------------------------- tensor maps (host)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time dependency on libcuda)
inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}
// bf16 matrix [rows, K] with row stride ld (elements); box = box_rows x 64 columns, 128-byte swizzle
inline bool make_map_2d(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t K, uint64_t ld, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[2] = {K, rows};
  cuuint64_t gstride[1] = {ld * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Rows of 128 bf16 seen as (64 elements, 2 halves, rows); a box is one half of box_rows consecutive rows.
inline bool make_map_rows128(CUtensorMap* m, const void* ptr, uint64_t rows, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[3] = {64, 2, rows};
  cuuint64_t gstride[2] = {128, 256};
  cuuint32_t box[3] = {64, 1, box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Rotated queries [rows, n_kv * rep * 128] bf16 seen as (64 elements, 2 halves, rep heads of a group, n_kv groups,
// rows): a box (64, 1, rep, 1, W) is one half of the W * rep query rows that share a KV head, in the row order
// (token, head) and with the 128-byte swizzle the tensor core reads.
inline bool make_map_q(CUtensorMap* m, const void* ptr, uint64_t rows, uint32_t rep, uint32_t n_kv, uint32_t W) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[5] = {64, 2, rep, n_kv, rows};
  cuuint64_t gstride[4] = {128, 256, static_cast<cuuint64_t>(rep) * 256, static_cast<cuuint64_t>(rep) * n_kv * 256};
  cuuint32_t box[5] = {64, 1, rep, 1, W};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
