// Part 1: greedy verify-accept and the row split (Section 2 "Preliminaries"; Algorithm 2
// "GreedyVerify"), plus the cos/sin tables of the positions this round touches.
#include "cod_internal.cuh"

// cos/sin of pos * theta^(-2j/hd) for the window rows (pos = L_s + p) and the next block's
// rows (pos = L_s + m_s + i). The angle is formed and reduced modulo 2*pi in double, so
// positions of tens of thousands lose nothing in float.
struct RopeTabs {
  const double* inv_freq;     // null: the verify kernel leaves the tables to k_rope_tables
  int half;
  float* rope_win;
  float* rope_blk;
};
__device__ __forceinline__ void rope_entry(const RopeTabs& t, int r, int j, int pos_win, int pos_blk) {
  const double two_pi = 6.283185307179586476925286766559;
  const double f = t.inv_freq[j];
  float sn, cs;
  if (t.rope_win) {
    double a = static_cast<double>(pos_win) * f;
    a -= two_pi * rint(a / two_pi);
    sincosf(static_cast<float>(a), &sn, &cs);
    t.rope_win[r * 2 * t.half + j] = cs; t.rope_win[r * 2 * t.half + t.half + j] = sn;
  }
  if (t.rope_blk) {
    double b = static_cast<double>(pos_blk) * f;
    b -= two_pi * rint(b / two_pi);
    sincosf(static_cast<float>(b), &sn, &cs);
    t.rope_blk[r * 2 * t.half + j] = cs; t.rope_blk[r * 2 * t.half + t.half + j] = sn;
  }
}
__global__ void k_rope_tables(const int32_t* __restrict__ committed_len, const int32_t* __restrict__ accept_len,
                              int S, int W, RopeTabs t) {
  cod_pdl_prologue();
  const int r = blockIdx.x, s = r / W, p = r - s * W;
  const int L = max(committed_len[s], 0);
  const int m = accept_len ? accept_len[s] : 0;
  for (int j = threadIdx.x; j < t.half; j += blockDim.x) rope_entry(t, r, j, L + p, L + m + p);
}

// One block. A warp handles one sequence at a time: each lane compares one window row,
// a ballot finds the first mismatch (acceptance is a PREFIX rule: a later match after the
// first mismatch does not count). Then a scan over sequences gives the CSR offsets and
// all threads write the per-row arrays (and, for small rounds, the cos/sin tables: one launch
// fewer at the head of the critical path).
__global__ void __launch_bounds__(1024)
k_verify_accept(const int32_t* __restrict__ draft, const int32_t* __restrict__ target, int S, int W,
                int n_forced, int vocab, int page, int max_pages, int n_pages,
                const int32_t* __restrict__ committed_len, const int32_t* __restrict__ block_table,
                cod_split out, uint32_t* status, const float* __restrict__ p_tok,
                const float* __restrict__ q_tok, const float* __restrict__ u, RopeTabs tabs) {
  cod_pdl_prologue();
  extern __shared__ int sm[];
  int* s_m = sm;              // [S]
  int* s_acc = sm + S;        // [S+1]
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  uint32_t flags = 0;

  for (int s = wid; s < S; s += nw) {
    int m = W;
    for (int p0 = 0; p0 < W && m == W; p0 += 32) {
      const int p = p0 + lane;
      bool ok = true;
      if (p < W) {
        if (p_tok == nullptr) {                       // greedy: the drafted token is the target's token
          const int d = draft[s * W + p], t = target[s * (W + 1) + p];
          if (d < 0 || d >= vocab || t < 0 || t >= vocab) flags |= COD_DEV_BAD_TOKEN;
          ok = (p < n_forced) || (d == t);
        } else {                                      // speculative sampling: accept with probability min(1, P/Q)
          ok = (p < n_forced) || (__fmul_rn(u[s * W + p], q_tok[s * W + p]) < p_tok[s * W + p]);
        }
      }
      const unsigned miss = __ballot_sync(0xffffffffu, !ok);
      if (miss) m = p0 + __ffs(miss) - 1;
    }
    if (lane == 0) {
      s_m[s] = m;
      int b = target[s * (W + 1) + m];
      if (b < 0 || b >= vocab) { flags |= COD_DEV_BAD_TOKEN; b = 0; }
      out.accept_len[s] = m;
      out.bonus[s] = b;
    }
  }
  __syncthreads();

  // exclusive prefix sums of m_s (warp 0, chunks of 32 with a running carry)
  if (wid == 0) {
    int run = 0;
    for (int s0 = 0; s0 < S; s0 += 32) {
      const int s = s0 + lane;
      const int v = s < S ? s_m[s] : 0;
      int inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      if (s < S) s_acc[s] = run + inc - v;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) s_acc[S] = run;
  }
  __syncthreads();

  for (int s = threadIdx.x; s <= S; s += blockDim.x) {
    out.acc_off[s] = s_acc[s];
    out.rej_off[s] = s * W - s_acc[s];
  }
  const int R = S * W, acc_total = s_acc[S];
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const int s = r / W, p = r - s * W, m = s_m[s];
    const int L = committed_len[s];
    if (L < 0) flags |= COD_DEV_BAD_LEN;
    const int pos = L + p;
    out.row_pos[r] = pos;
    int cslot = -1, uslot = -1;
    if (p < m) {
      const int lp = pos / page;
      if (L < 0 || lp >= max_pages) {
        flags |= COD_DEV_PAGE_OVERFLOW;
      } else {
        const int pg = block_table[s * max_pages + lp];
        if (pg < 0 || pg >= n_pages) flags |= COD_DEV_BAD_PAGE;
        else cslot = pg * page + pos % page;
      }
      out.acc_rows[s_acc[s] + p] = r;
    } else {
      uslot = s * W + (p - m);
      out.rej_rows[(s * W - s_acc[s]) + (p - m)] = r;
    }
    out.commit_slot[r] = cslot;
    out.carry_slot[r] = uslot;
    if (r >= acc_total) out.acc_rows[r] = -1;
    if (r >= R - acc_total) out.rej_rows[r] = -1;
  }
  if (flags) atomicOr(status, flags);
  if (tabs.inv_freq != nullptr)
    for (int e = threadIdx.x; e < R * tabs.half; e += blockDim.x) {
      const int r = e / tabs.half, j = e - r * tabs.half, s = r / W, p = r - s * W;
      const int L = max(committed_len[s], 0);
      rope_entry(tabs, r, j, L + p, L + s_m[s] + p);
    }
}

int cod_launch_verify(cod_ctx* c, const int32_t* draft, const int32_t* target, int S, int n_forced,
                      const cod_state* state, const cod_split* out, cudaStream_t st, const float* p_tok,
                      const float* q_tok, const float* u) {
  ProfScope prof(c, COD_K_VERIFY, st);
  const int W = c->cfg.block;
  const size_t smem = static_cast<size_t>(2 * S + 2) * sizeof(int);
  const RopeTabs tabs{c->inv_freq_d, c->half, c->rope_win, c->rope_blk};
  const bool fold = S * W * c->half <= 4096;        // a few table entries per thread at most
  cod_launch_pdl(c, k_verify_accept, 1, 1024, smem, st, draft, target, S, W, n_forced, c->cfg.vocab, c->cfg.page_size,
                                         c->cfg.max_pages_per_seq, c->cfg.n_pages, state->committed_len,
                                         state->block_table, *out, c->status, p_tok, q_tok, u,
                                         fold ? tabs : RopeTabs{nullptr, 0, nullptr, nullptr});
  COD_CHECK_LAUNCH(c);
  if (!fold) {
    cod_launch_pdl(c, k_rope_tables, S * W, 64, 0, st, state->committed_len, out->accept_len, S, W, tabs);
    COD_CHECK_LAUNCH(c);
  }
  return COD_OK;
}

int cod_launch_rope_blk_only(cod_ctx* c, const int32_t* committed_len, int S, cudaStream_t st) {
  ProfScope prof(c, COD_K_VERIFY, st);
  cod_launch_pdl(c, k_rope_tables, S * c->cfg.block, 64, 0, st, committed_len, nullptr, S, c->cfg.block,
                 RopeTabs{c->inv_freq_d, c->half, nullptr, c->rope_blk});
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

// Re-convergence count of Section 5.2: one warp per sequence, a lane per rejected position.
__global__ void k_reconvergence(const int32_t* __restrict__ z, const int32_t* __restrict__ y,
                                const int32_t* __restrict__ len, int S, int W, int32_t* __restrict__ R) {
  cod_pdl_prologue();
  const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (s >= S) return;
  const int L = min(max(len[s], 0), W);
  int cnt = 0;
  for (int q = lane; q < L; q += 32) {
    const int t = y[s * W + q];
    bool hit = z[s * W + q] == t;
    if (q > 0) hit = hit || z[s * W + q - 1] == t;
    if (q + 1 < L) hit = hit || z[s * W + q + 1] == t;
    cnt += hit ? 1 : 0;
  }
  for (int o = 16; o >= 1; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if (lane == 0) R[s] = cnt;
}

int cod_launch_reconvergence(cod_ctx* c, const int32_t* z, const int32_t* y, const int32_t* len, int S,
                             int32_t* R, cudaStream_t st) {
  ProfScope prof(c, COD_K_VERIFY, st);
  cod_launch_pdl(c, k_reconvergence, (S + 3) / 4, 128, 0, st, z, y, len, S, c->cfg.block, R);
  COD_CHECK_LAUNCH(c);
  return COD_OK;
}

