"""CPU oracle of one Carryover drafting round.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy statement of what the round computes, written from
the paper (Section 2 "Carryover Drafting", Eq. 1, Eq. 2; Appendix A, Algorithm 1
and its "Cache semantics" paragraph).  It exists to check the CUDA library; it
shares no code with it and is never on the product path: only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.

Every part below has an exact definition (a prefix rule on integers, linear
maps, a plane rotation, softmax attention, an argmax), so the oracle is that
definition written out: no tiling, no online softmax, no fused steps.  numpy's
``@`` (a library matmul in float64) serves as the contraction step.

Where the paper leaves the drafter body open (the equations "omit attention
normalisation and positional encoding", Section 2.1), the readings taken are:
  * F, K_l, V_l, W_q, W_o are bias-free linear maps stored [out, in];
  * an RMS normalisation with gain follows F (switchable), precedes each
    attention sub-layer, and precedes the LM head; the residual stream is
    x <- x + W_o o; by default there is no MLP;
  * the complete layer (d_ff > 0, qk_norm; the shape of the Qwen3 blocks the
    paper's DFlash drafters are built from, Section 4 "Targets and drafters")
    adds a per-head RMS norm with gain on queries and on ALL keys (cached and
    block keys alike) before the rotation, and after the attention residual
    x <- x + W_down( silu(W_gate b) * (W_up b) ) with b = N(x) * g_mlp;
  * RoPE is the rotate-half form over the full head dimension, at the absolute
    token position, applied once to keys when they are projected (Appendix A,
    "Cache semantics") and to the block's queries and keys at draft time;
  * the block is [bonus token, MASK, ..., MASK]; every block query sees all
    committed rows, all carried rows and all block rows (no mask), scale
    1/sqrt(hd); grouped-query attention maps query head g to KV head
    g // (n_q / n_kv);
  * the LM head is the transposed embedding table; argmax ties go to the lowest id.

Two ways to run it.  Exact (the default, and the only truth any tolerance is
judged against): float64 everywhere on the given inputs.  Storage-rounded (a
DIAGNOSTIC, never the pass/fail truth): the same steps with a caller-supplied
``round_store`` applied wherever an implementation that keeps bfloat16 tensors
between its steps would store one (the fused features z, cached K/V, normalised
activations, the block's rotated q/k and v, attention outputs, MLP activations,
the LM head's input); it separates storage noise from a real defect when an
error sits near a bound.  With ``round_store=None`` no arithmetic changes.

Parity status: every function here is pinned by tests/test_oracle_pins.py
against closed forms, brute force, invariants the paper states, and library
special cases (the drafter pass's attention sub-layer by a hand-written layer
and by torch linear / rms_norm).  What stays unpinned is the choice of the readings above
themselves: the paper ships no reference numbers for this path, so they are
pinned to their written definition only ("parity unpinned" against the authors'
system for the drafter-body glue).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

MODE_CARRY = 0      # Algorithm 1, right column
MODE_BASELINE = 1   # Algorithm 1, left column


@dataclass
class OracleConfig:
    d_target: int
    n_cap: int
    d_model: int
    n_layers: int
    n_q: int
    n_kv: int
    hd: int
    vocab: int
    mask_token_id: int
    W: int
    page: int
    rope_theta: float
    rms_eps: float
    hidden_norm: bool
    d_ff: int = 0            # > 0: every drafter layer has a gated MLP of this width
    qk_norm: bool = False    # per-head RMS norm of queries and keys before the rotation
    carry_rounds: int = 1    # k: rejected rows are retained for k rounds (the paper uses and trains k = 1;
                             # Section 6 names retention beyond one round as what different rollouts would allow)
    carry_variant: str = "embedding"   # "embedding": E_carry on rejected rows (Eq. 2, the paper's choice);
                                       # "none": rejected rows pass F unmarked; "projector": rejected rows
                                       # pass their own fusion map F_rej (Table 4(b)'s two alternatives)

    @property
    def d_in(self) -> int:
        return self.d_target * self.n_cap


def prepare_weights(weights: Dict[str, np.ndarray]) -> Dict[str, np.ndarray]:
    """float64 copies of the weight arrays (made once; the values are unchanged)."""
    return {k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}


class OracleState:
    """Committed drafter KV C_l (paged), carried KV U_l, and their lengths.

    pool  [Ld, n_pages, n_kv, 2, page, hd]   index 3: 0 = K (already rotated), 1 = V
    carry [Ld, S, n_kv, 2, k*W, hd]          rows >= carry_len[s] are NaN (never to be read)
    carry_hist[s]                            lengths of the (at most k) rounds' segments held in U, oldest first
    """

    def __init__(self, cfg: OracleConfig, S: int, n_pages: int, block_table: np.ndarray,
                 committed_len: np.ndarray):
        self.cfg = cfg
        self.S = S
        self.pool = np.zeros((cfg.n_layers, n_pages, cfg.n_kv, 2, cfg.page, cfg.hd), dtype=np.float64)
        self.block_table = np.array(block_table, dtype=np.int64)
        self.committed_len = np.array(committed_len, dtype=np.int64)
        self.carry = np.full((cfg.n_layers, S, cfg.n_kv, 2, cfg.carry_rounds * cfg.W, cfg.hd), np.nan, dtype=np.float64)
        self.carry_hist = [[] for _ in range(S)]
        # Algorithm 1: "Initialize U_l = empty".
        self.carry_len = np.zeros(S, dtype=np.int64)


# =========================================================================== part 1
def verify_accept(draft: np.ndarray, target: np.ndarray, committed_len: np.ndarray,
                  block_table: np.ndarray, page: int, n_forced: int) -> Dict[str, np.ndarray]:
    """Greedy verification (Section 2, "Preliminaries"; Algorithm 2 "GreedyVerify").

    The target accepts the longest PREFIX of the window whose tokens equal its own
    greedy tokens; rejection stops acceptance of the whole suffix (Appendix B.1).
    target[s, p] is the target's greedy token for window row p (W+1 entries), so the
    token after the accepted prefix, target[s, m], is the bonus token.  The first
    n_forced rows (the anchor) count as accepted whatever they hold.

    Rows p < m are accepted (H^acc), rows p >= m are rejected (H^rej), Eq. 1.  Row p
    sits at absolute position L_s + p ("each rejected state keeps the absolute
    position of the token at which it was computed").
    """
    draft = np.asarray(draft)
    target = np.asarray(target)
    S, W = draft.shape
    accept_len = np.zeros(S, dtype=np.int32)
    bonus = np.zeros(S, dtype=np.int32)
    row_pos = np.zeros(S * W, dtype=np.int32)
    commit_slot = np.full(S * W, -1, dtype=np.int32)
    carry_slot = np.full(S * W, -1, dtype=np.int32)
    acc_rows, rej_rows = [], []
    acc_off, rej_off = [0], [0]
    for s in range(S):
        m = 0
        while m < W and (m < n_forced or int(draft[s, m]) == int(target[s, m])):
            m += 1
        accept_len[s] = m
        bonus[s] = target[s, m]
        L = int(committed_len[s])
        for p in range(W):
            row = s * W + p
            pos = L + p
            row_pos[row] = pos
            if p < m:
                commit_slot[row] = int(block_table[s, pos // page]) * page + pos % page
                acc_rows.append(row)
            else:
                carry_slot[row] = s * W + (p - m)
                rej_rows.append(row)
        acc_off.append(len(acc_rows))
        rej_off.append(len(rej_rows))
    pad = lambda lst: np.array(lst + [-1] * (S * W - len(lst)), dtype=np.int32)
    return {
        "accept_len": accept_len, "bonus": bonus, "row_pos": row_pos,
        "commit_slot": commit_slot, "carry_slot": carry_slot,
        "acc_rows": pad(acc_rows), "acc_off": np.array(acc_off, dtype=np.int32),
        "rej_rows": pad(rej_rows), "rej_off": np.array(rej_off, dtype=np.int32),
    }


def verify_accept_stochastic(p_tok: np.ndarray, q_tok: np.ndarray, u: np.ndarray, target: np.ndarray,
                             committed_len: np.ndarray, block_table: np.ndarray, page: int,
                             n_forced: int) -> Dict[str, np.ndarray]:
    """Speculative-sampling verification (Appendix A, "Why verification remains valid": the usual
    target acceptance and residual correction applied with the drafter's actual proposal
    distribution q).

    Row p of the window is accepted with probability min(1, P(x_p) / Q(x_p)), x_p the drafted
    token, and acceptance is again a PREFIX rule: the first rejected row ends it.  Inputs are the two
    probabilities of the drafted token and a uniform number per row; the decision is
    u * q < p, taken in float32 (one rounded product and a comparison, so every implementation
    takes the same decision).  target[s, m] is the token the target's sampler supplies after the
    accepted prefix: drawn from the residual norm(max(0, P - Q)) at the first rejected row, or
    from P after a fully accepted window.  Everything downstream (row split, slots) is as in
    verify_accept.
    """
    p32 = np.asarray(p_tok, dtype=np.float32)
    q32 = np.asarray(q_tok, dtype=np.float32)
    u32 = np.asarray(u, dtype=np.float32)
    S, W = p32.shape
    ok = (u32 * q32) < p32                       # float32 product, rounded once
    # express the rule through the greedy routine: a window whose "draft" equals the "target"
    # exactly on the rows the coin accepted
    fake_target = np.array(target, dtype=np.int64)
    fake_draft = np.where(ok, fake_target[:, :W], fake_target[:, :W] + 1)
    return verify_accept(fake_draft, fake_target, committed_len, block_table, page, n_forced)


# =========================================================================== shared pieces
def rope(x: np.ndarray, pos, theta: float) -> np.ndarray:
    """Rotate-half rotary embedding of x[..., hd] at absolute position(s) pos.

    Pair (j, j + hd/2) is rotated by the angle pos * theta^(-2j/hd).
    pos broadcasts against x[..., 0].
    """
    x = np.asarray(x, dtype=np.float64)
    hd = x.shape[-1]
    half = hd // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = np.float64(theta) ** (-2.0 * j / hd)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """g * x / sqrt(mean(x^2) + eps) over the last axis."""
    x = np.asarray(x, dtype=np.float64)
    return g * x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)


def silu(x: np.ndarray) -> np.ndarray:
    """x * sigmoid(x)."""
    x = np.asarray(x, dtype=np.float64)
    return x / (1.0 + np.exp(-x))


def gated_mlp(b: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, w_down: np.ndarray) -> np.ndarray:
    """W_down( silu(W_gate b) * (W_up b) ) for rows b [R, D]; matrices stored [out, in]."""
    return (silu(b @ w_gate.T) * (b @ w_up.T)) @ w_down.T


# =========================================================================== part 2
def fuse_features(H: np.ndarray, rejected: np.ndarray, w: Dict[str, np.ndarray],
                  cfg: OracleConfig) -> np.ndarray:
    """Z = F(H^keep) with E_carry added to the rejected rows first (Eq. 2; Algorithm 1
    right column, steps 2-3: the embedding is added "before projection by F")."""
    Hk = np.asarray(H, dtype=np.float64).copy()
    if cfg.carry_variant == "embedding":
        Hk[rejected] = Hk[rejected] + w["e_carry"]
    Z = Hk @ w["fc"].T
    if cfg.carry_variant == "projector":
        # Section 5 "How should rejected states be distinguished?": a separate projector for the
        # rejected rows instead of the embedding (its shape is not given; taken as F's)
        Z[rejected] = Hk[rejected] @ w["fc_rej"].T
    if cfg.hidden_norm:
        Z = rmsnorm(Z, w["g_hidden"], cfg.rms_eps)
    return Z


def _stored(x: np.ndarray, round_store) -> np.ndarray:
    """x as an implementation with reduced-precision storage would hold it (diagnostic mode only)."""
    return x if round_store is None else np.asarray(round_store(x), dtype=np.float64)


def project_kv(H: np.ndarray, split: Dict[str, np.ndarray], w: Dict[str, np.ndarray],
               cfg: OracleConfig, mode: int, round_store=None) -> np.ndarray:
    """J_l = (K_l(Z), V_l(Z)) for every drafter layer (Eq. 1; Algorithm 1 step "J_l").

    Carry mode keeps all window rows; baseline mode keeps the accepted rows only
    (the others come back as NaN: they do not exist in that column of Algorithm 1).
    Keys are rotated at their row's absolute position.  Output [Ld, R, 2, n_kv, hd].
    """
    R = H.shape[0]
    W = cfg.W
    m_of_row = np.repeat(np.asarray(split["accept_len"], dtype=np.int64), W)
    p_of_row = np.tile(np.arange(W), R // W)
    rejected = p_of_row >= m_of_row
    keep = np.ones(R, dtype=bool) if mode == MODE_CARRY else ~rejected
    Z = _stored(fuse_features(H, rejected, w, cfg), round_store)
    J = np.full((cfg.n_layers, R, 2, cfg.n_kv, cfg.hd), np.nan, dtype=np.float64)
    pos = np.asarray(split["row_pos"], dtype=np.float64)
    for l in range(cfg.n_layers):
        K = (Z @ w["wk"][l].T).reshape(R, cfg.n_kv, cfg.hd)
        V = (Z @ w["wv"][l].T).reshape(R, cfg.n_kv, cfg.hd)
        if cfg.qk_norm:
            K = rmsnorm(K, w["g_knorm"][l], cfg.rms_eps)
        K = _stored(rope(K, pos[:, None], cfg.rope_theta), round_store)
        V = _stored(V, round_store)
        J[l, keep, 0] = K[keep]
        J[l, keep, 1] = V[keep]
    return J


# =========================================================================== part 3
def scatter_kv(J: np.ndarray, split: Dict[str, np.ndarray], st: OracleState, mode: int) -> None:
    """C_l <- [C_l; J_{l,1:m}],  U_l <- J_{l,m+1:B} replacing the old U_l (Algorithm 1,
    right column, last three steps); the baseline column appends only and leaves U empty."""
    cfg = st.cfg
    W, page = cfg.W, cfg.page
    for s in range(st.S):
        m = int(split["accept_len"][s])
        L = int(st.committed_len[s])
        for l in range(cfg.n_layers):
            for p in range(m):
                pos = L + p
                pg = int(st.block_table[s, pos // page])
                st.pool[l, pg, :, 0, pos % page, :] = J[l, s * W + p, 0]
                st.pool[l, pg, :, 1, pos % page, :] = J[l, s * W + p, 1]
            if mode != MODE_CARRY:
                st.carry[l, s] = np.nan                   # the baseline column keeps no U at all
        if mode == MODE_CARRY:
            # U holds the rejected rows of the last k rounds, oldest first (k = 1: "U_l <- J_l rejected",
            # the previous U discarded). A round that rejects nothing still ages the older segments.
            c_old = int(st.carry_len[s])
            hist = st.carry_hist[s][-(cfg.carry_rounds - 1):] if cfg.carry_rounds > 1 else []
            keep = sum(hist)                              # rows of the k - 1 newest rounds, at the end of U
            drop = c_old - keep
            st.carry_hist[s] = hist + [W - m]
            for l in range(cfg.n_layers):
                kept = st.carry[l, s, :, :, drop:c_old, :].copy()
                st.carry[l, s] = np.nan
                st.carry[l, s, :, :, :keep, :] = kept
                for p in range(m, W):
                    st.carry[l, s, :, 0, keep + p - m, :] = J[l, s * W + p, 0]
                    st.carry[l, s, :, 1, keep + p - m, :] = J[l, s * W + p, 1]
            st.carry_len[s] = keep + (W - m)
        else:
            st.carry_hist[s] = []
            st.carry_len[s] = 0
        st.committed_len[s] = L + m


# =========================================================================== part 4
def gather_ctx(st: OracleState, layer: int, s: int, use_carry: bool):
    """ctx_l = [C_l; U_l] of sequence s as dense arrays K, V [n_kv, L' + c, hd] (Eq. 2)."""
    cfg = st.cfg
    L = int(st.committed_len[s])
    t = np.arange(L)
    pages = st.block_table[s, t // cfg.page]
    Kc = st.pool[layer, pages, :, 0, t % cfg.page, :]      # [L, n_kv, hd]
    Vc = st.pool[layer, pages, :, 1, t % cfg.page, :]
    K = np.transpose(Kc, (1, 0, 2))
    V = np.transpose(Vc, (1, 0, 2))
    c = int(st.carry_len[s]) if use_carry else 0
    if c > 0:
        K = np.concatenate([K, st.carry[layer, s, :, 0, :c, :]], axis=1)
        V = np.concatenate([V, st.carry[layer, s, :, 1, :c, :]], axis=1)
    return K, V, c


def block_attn(layer: int, q: np.ndarray, k_blk: np.ndarray, v_blk: np.ndarray,
               st: OracleState, use_carry: bool, round_store=None):
    """Block attention over [C_l; U_l; block] (Section 2 "Preliminaries": draft positions
    attend to the keys and values made from target hidden states; Algorithm 1: "the next
    draft reads ctx_l").

    q [S, W, n_q, hd], k_blk / v_blk [S, W, n_kv, hd], q and k_blk NOT yet rotated: block
    row i of sequence s sits at position L'_s + i.  Returns out [S, W, n_q, hd] and the
    softmax mass that falls on the carried rows [S, W, n_q] (Appendix C's diagnostic).
    """
    cfg = st.cfg
    S, W = q.shape[0], q.shape[1]
    rep = cfg.n_q // cfg.n_kv
    out = np.zeros((S, W, cfg.n_q, cfg.hd), dtype=np.float64)
    mass = np.zeros((S, W, cfg.n_q), dtype=np.float64)
    for s in range(S):
        L = int(st.committed_len[s])
        pos = (L + np.arange(W)).astype(np.float64)
        qr = _stored(rope(np.asarray(q[s], dtype=np.float64), pos[:, None], cfg.rope_theta), round_store)
        kr = _stored(rope(np.asarray(k_blk[s], dtype=np.float64), pos[:, None], cfg.rope_theta), round_store)
        vr = _stored(np.asarray(v_blk[s], dtype=np.float64), round_store)
        Kctx, Vctx, c = gather_ctx(st, layer, s, use_carry)
        K = np.concatenate([Kctx, np.transpose(kr, (1, 0, 2))], axis=1)        # [n_kv, T, hd]
        V = np.concatenate([Vctx, np.transpose(vr, (1, 0, 2))], axis=1)
        for g in range(cfg.n_q):
            h = g // rep
            sc = (qr[:, g, :] @ K[h].T) / np.sqrt(np.float64(cfg.hd))          # [W, T]
            sc = sc - sc.max(axis=1, keepdims=True)
            pr = np.exp(sc)
            pr = pr / pr.sum(axis=1, keepdims=True)
            out[s, :, g, :] = pr @ V[h]
            mass[s, :, g] = pr[:, L:L + c].sum(axis=1)
    return _stored(out, round_store), mass


# =========================================================================== part 5
def lm_head_argmax(x: np.ndarray, w: Dict[str, np.ndarray], cfg: OracleConfig, round_store=None):
    """logits = N_f(x) Emb^T; token = lowest-index argmax; also the top-2 logit gap."""
    y = _stored(rmsnorm(x, w["g_final"], cfg.rms_eps), round_store)
    logits = y @ w["emb"].T
    tok = np.argmax(logits, axis=1).astype(np.int32)          # first occurrence = lowest id
    top2 = np.partition(logits, -2, axis=1)[:, -2:]
    gap = top2[:, 1] - top2[:, 0]
    return tok, gap, logits


def lm_head_rank(x: np.ndarray, ref_tok: np.ndarray, w: Dict[str, np.ndarray], cfg: OracleConfig,
                 tol: float = 0.0, round_act=None):
    """Rank of a reference token among the drafter's candidates (Section 5.1 "Target-token recall at
    matched anchors": Recall@k asks whether the target's top token is among the drafter's k best, i.e.
    whether this rank is below k).  rank[r] = number of vocabulary entries v != ref_tok[r] whose logit
    N_f(x[r]) . Emb[v] is above the reference token's, ties going to the lower index.

    Returns (rank, ref_logit, rank_lo, rank_hi): rank_lo / rank_hi count the entries above
    ref_logit + tol resp. above ref_logit - tol, the window inside which an implementation in other
    arithmetic may legitimately land.  A rank is an integer decided by floating point: round_act
    (default none), applied to the normalised activations, lets a test take that decision in the
    operand precision of the implementation it checks (e.g. rounding to bfloat16)."""
    y = rmsnorm(x, w["g_final"], cfg.rms_eps)
    if round_act is not None:
        y = round_act(y)
    logits = y @ w["emb"].T
    R, V = logits.shape
    ref_tok = np.asarray(ref_tok, dtype=np.int64)
    ref = logits[np.arange(R), ref_tok]
    idx = np.arange(V)[None, :]
    other = idx != ref_tok[:, None]
    above = (logits > ref[:, None]) | ((logits == ref[:, None]) & (idx < ref_tok[:, None]))
    rank = (above & other).sum(axis=1).astype(np.int32)
    rank_lo = ((logits > ref[:, None] + tol) & other).sum(axis=1).astype(np.int32)
    rank_hi = ((logits > ref[:, None] - tol) & other).sum(axis=1).astype(np.int32)
    return rank, ref, rank_lo, rank_hi


# --------------------------------------------------------------------------- sampling head
def counter_uniform(seed: int, step: int, row: np.ndarray, col: np.ndarray) -> np.ndarray:
    """The counter-based uniform number U(seed, step, row, col) in (0, 1) both sides draw for the
    Gumbel-max sample of the LM head (the paper fixes no generator; this one is the reading taken).

    A 32-bit integer hash: h = mix(mix(mix(seed_lo ^ K0) + seed_hi) + step) ... of the four counters
    chained through the 'murmur3 finaliser' mix(x): x ^= x >> 16; x *= 0x85EBCA6B; x ^= x >> 13;
    x *= 0xC2B2AE35; x ^= x >> 16 (all modulo 2^32).  U = ((h >> 9) + 0.5) * 2^-23 = (2k + 1) / 2^24, exactly
    representable in float32.
    """
    M = np.uint64(0xFFFFFFFF)

    def mix(x):
        x = x & M
        x ^= x >> np.uint64(16)
        x = (x * np.uint64(0x85EBCA6B)) & M
        x ^= x >> np.uint64(13)
        x = (x * np.uint64(0xC2B2AE35)) & M
        x ^= x >> np.uint64(16)
        return x

    seed = int(seed)
    h = mix(np.uint64((seed & 0xFFFFFFFF) ^ 0x9E3779B9))
    h = mix((h + np.uint64((seed >> 32) & 0xFFFFFFFF)) & M)
    h = mix((h + np.uint64(int(step) & 0xFFFFFFFF)) & M)
    h = mix((h + np.asarray(row, dtype=np.uint64)) & M)
    h = mix((h + np.asarray(col, dtype=np.uint64)) & M)
    return ((h >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def lm_head_sample(x: np.ndarray, w: Dict[str, np.ndarray], cfg: OracleConfig, seed: int, step: int,
                   row_ids: Optional[np.ndarray] = None):
    """A token per row drawn from softmax(N_f(x) Emb^T) by the Gumbel-max rule:
    tok = argmax_v (logit_v - log(-log U_v)), lowest index on ties, U from counter_uniform with
    row = the row index and col = the token id.  Returns tok, q_tok = softmax(logits)[tok],
    the log-sum-exp of the logits and the top-2 gap of the PERTURBED logits (near-ties may
    legitimately fall either way on another implementation).  row_ids (default 0..R-1) are the
    row counters of the noise, for callers that pass a subset of a larger batch's rows."""
    y = rmsnorm(x, w["g_final"], cfg.rms_eps)
    logits = y @ w["emb"].T
    R, V = logits.shape
    rows = np.arange(R) if row_ids is None else np.asarray(row_ids)
    U = counter_uniform(seed, step, rows[:, None], np.arange(V)[None, :])
    pert = logits - np.log(-np.log(U))
    tok = np.argmax(pert, axis=1).astype(np.int32)
    mx = logits.max(axis=1)
    lse = mx + np.log(np.exp(logits - mx[:, None]).sum(axis=1))
    q_tok = np.exp(logits[np.arange(R), tok] - lse)
    top2 = np.partition(pert, -2, axis=1)[:, -2:]
    return tok, q_tok, lse, top2[:, 1] - top2[:, 0]


# =========================================================================== the drafter pass
def draft_block(st: OracleState, bonus: np.ndarray, w: Dict[str, np.ndarray],
                use_carry: bool, keep_logits: bool = False, round_store=None) -> Dict[str, np.ndarray]:
    """One parallel block prediction from [bonus, MASK, ...] reading ctx_l in every layer."""
    cfg = st.cfg
    S, W, D = st.S, cfg.W, cfg.d_model
    toks = np.full((S, W), cfg.mask_token_id, dtype=np.int64)
    toks[:, 0] = bonus
    x = w["emb"][toks.reshape(-1)].copy()                                     # [R, D]
    attn_out = np.zeros((cfg.n_layers, S * W, cfg.n_q * cfg.hd), dtype=np.float64)
    mass = np.zeros((cfg.n_layers, S, W, cfg.n_q), dtype=np.float64)
    for l in range(cfg.n_layers):
        a = _stored(rmsnorm(x, w["g_attn"][l], cfg.rms_eps), round_store)
        q = (a @ w["wq"][l].T).reshape(S, W, cfg.n_q, cfg.hd)
        kb = (a @ w["wk"][l].T).reshape(S, W, cfg.n_kv, cfg.hd)
        vb = (a @ w["wv"][l].T).reshape(S, W, cfg.n_kv, cfg.hd)
        if cfg.qk_norm:
            q = rmsnorm(q, w["g_qnorm"][l], cfg.rms_eps)
            kb = rmsnorm(kb, w["g_knorm"][l], cfg.rms_eps)
        o, mass[l] = block_attn(l, q, kb, vb, st, use_carry, round_store)
        attn_out[l] = o.reshape(S * W, cfg.n_q * cfg.hd)
        x = x + attn_out[l] @ w["wo"][l].T
        if cfg.d_ff > 0:
            b = _stored(rmsnorm(x, w["g_mlp"][l], cfg.rms_eps), round_store)
            if round_store is None:
                x = x + gated_mlp(b, w["w_gate"][l], w["w_up"][l], w["w_down"][l])
            else:                                         # the gated activation is a stored tensor too
                act = _stored(silu(b @ w["w_gate"][l].T) * (b @ w["w_up"][l].T), round_store)
                x = x + act @ w["w_down"][l].T
    tok, gap, logits = lm_head_argmax(x, w, cfg, round_store)
    res = {"tok": tok.reshape(S, W), "gap": gap.reshape(S, W), "x_final": x,
           "attn_out": attn_out, "carry_mass": mass}
    if keep_logits:
        res["logits"] = logits
    return res


def draft_round(draft: np.ndarray, target: np.ndarray, H: np.ndarray, st: OracleState,
                w: Dict[str, np.ndarray], n_forced: int, mode: int,
                keep_logits: bool = False, round_store=None) -> Dict[str, np.ndarray]:
    """verify-accept -> project -> scatter -> draft the next block (Algorithm 1, then
    "the next draft reads ctx_l").  Mutates st.  next_draft = [bonus, tok_1 .. tok_{W-1}]."""
    cfg = st.cfg
    split = verify_accept(draft, target, st.committed_len, st.block_table, cfg.page, n_forced)
    J = project_kv(H, split, w, cfg, mode, round_store)
    scatter_kv(J, split, st, mode)
    res = draft_block(st, split["bonus"], w, use_carry=(mode == MODE_CARRY), keep_logits=keep_logits,
                      round_store=round_store)
    next_draft = res["tok"].copy()
    next_draft[:, 0] = split["bonus"]
    res.update(split=split, J=J, next_draft=next_draft.astype(np.int32))
    return res


def draft_round_stochastic(target: np.ndarray, p_tok: np.ndarray, q_tok: np.ndarray, u: np.ndarray,
                           H: np.ndarray, st: OracleState, w: Dict[str, np.ndarray], n_forced: int,
                           mode: int, sample: Optional[tuple] = None) -> Dict[str, np.ndarray]:
    """draft_round with speculative-sampling verification as its first step (Appendix A, "Why
    verification remains valid": Carryover changes the proposal distribution, not the rule).
    sample = (seed, step): the next block is drawn by lm_head_sample (row counters 0..R-1) instead
    of taken greedily; the result then also holds q_next and the perturbed top-2 gap."""
    cfg = st.cfg
    split = verify_accept_stochastic(p_tok, q_tok, u, target, st.committed_len, st.block_table, cfg.page, n_forced)
    J = project_kv(H, split, w, cfg, mode)
    scatter_kv(J, split, st, mode)
    res = draft_block(st, split["bonus"], w, use_carry=(mode == MODE_CARRY))
    if sample is not None:
        tok, q, _, gap = lm_head_sample(res["x_final"], w, cfg, sample[0], sample[1])
        res["tok"] = tok.reshape(st.S, cfg.W)
        res["gap"] = gap.reshape(st.S, cfg.W)
        res["q_next"] = q.reshape(st.S, cfg.W)
    next_draft = res["tok"].copy()
    next_draft[:, 0] = split["bonus"]
    res.update(split=split, J=J, next_draft=next_draft.astype(np.int32))
    return res


# =========================================================================== analysis aids
def reconvergence_count(z: np.ndarray, y: np.ndarray, length: np.ndarray) -> np.ndarray:
    """Re-convergence count R of Section 5.2 ("Why do gains differ across datasets?", the
    equation defining R), per sequence.

    z[s, q]: the verifier's top-1 next-token prediction from the q-th rejected state;
    y[s, q]: the token eventually committed at the position that prediction refers to;
    length[s]: the rejected suffix length L.  Position q counts if z_{q+d} = y_q for some
    d in {-1, 0, +1}, indices outside [0, L) ignored (a one-position tolerance for a local
    insertion or deletion).
    """
    z = np.asarray(z)
    y = np.asarray(y)
    S = z.shape[0]
    out = np.zeros(S, dtype=np.int32)
    for s in range(S):
        L = int(length[s])
        for q in range(L):
            hit = False
            for d in (-1, 0, 1):
                if 0 <= q + d < L and int(z[s, q + d]) == int(y[s, q]):
                    hit = True
            out[s] += 1 if hit else 0
    return out

