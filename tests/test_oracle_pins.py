"""Pins for the CPU oracle: each part is checked against something other than itself —
closed forms, brute force on tiny inputs, invariants the paper states (Section 2.1 and
Appendix A "Cache semantics"), and library routines it must reduce to.

The paper prints no worked numeric example for the drafting round (all of its numbers
need trained checkpoints), so there is no table of printed values to compare with; see
tests/golden/README.md.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import cod_oracle as orc
from paper_2609_14717_b200 import synth
from tests.helpers import oracle_config, oracle_state, small_bf16


# ----------------------------------------------------------------------------- part 1
def _first_zero(bits):
    """Index of the first False in a tuple of booleans (len if none) — via string search."""
    s = "".join("1" if b else "0" for b in bits)
    i = s.find("0")
    return len(s) if i < 0 else i


@pytest.mark.parametrize("n_forced", [0, 1])
def test_accept_is_prefix_rule_exhaustive_W8(n_forced):
    W, page = 8, 16
    pats = list(itertools.product([False, True], repeat=W))
    S = len(pats)
    rng = np.random.default_rng(1)
    draft = rng.integers(0, 50, size=(S, W)).astype(np.int32)
    target = rng.integers(0, 50, size=(S, W + 1)).astype(np.int32)
    for s, bits in enumerate(pats):
        for p, b in enumerate(bits):
            target[s, p] = draft[s, p] if b else draft[s, p] + 100   # mismatch for certain
    L = rng.integers(0, 100, size=S).astype(np.int32)
    bt = rng.permutation(S * 8).reshape(S, 8).astype(np.int32)
    out = orc.verify_accept(draft, target, L, bt, page, n_forced)
    for s, bits in enumerate(pats):
        eff = tuple(b or p < n_forced for p, b in enumerate(bits))
        m = _first_zero(eff)
        assert out["accept_len"][s] == m                      # a later match never counts
        assert out["bonus"][s] == target[s, m]
    # counts and offsets
    assert out["acc_off"][-1] + out["rej_off"][-1] == S * W
    assert np.array_equal(np.diff(out["acc_off"]), out["accept_len"])
    assert np.array_equal(np.diff(out["rej_off"]), W - out["accept_len"])
    # lists are the row ids in increasing order, split by acceptance
    acc = out["acc_rows"][:out["acc_off"][-1]]
    rej = out["rej_rows"][:out["rej_off"][-1]]
    assert np.all(np.diff(acc) > 0) and np.all(np.diff(rej) > 0)
    assert sorted(list(acc) + list(rej)) == list(range(S * W))
    # slots by the direct formula
    for row in range(S * W):
        s, p = divmod(row, W)
        pos = int(L[s]) + p
        assert out["row_pos"][row] == pos
        if p < out["accept_len"][s]:
            assert out["commit_slot"][row] == bt[s, pos // page] * page + pos % page
            assert out["carry_slot"][row] == -1
        else:
            assert out["commit_slot"][row] == -1
            assert out["carry_slot"][row] == s * W + p - out["accept_len"][s]


@pytest.mark.parametrize("name", ["cfg1", "cfg3"])
def test_accept_matches_generator_intent(name):
    """The token generator builds draft/target to realise a chosen m; the oracle must find it."""
    wl = synth.workload(name)
    lay = synth.make_layout(wl, 3)
    for r in range(8):
        rng = np.random.default_rng([3, 99, r])
        m = synth.draw_accept(wl, rng)
        draft, target = synth.make_tokens(wl, rng, m)
        out = orc.verify_accept(draft, target, lay["committed_len"], lay["block_table"],
                                wl.shape.page, wl.n_forced)
        assert np.array_equal(out["accept_len"], m)
        assert 0 <= (wl.shape.W - out["accept_len"]).max() <= wl.shape.W


def test_forced_anchor_row_is_accepted_even_if_tokens_differ():
    draft = np.array([[5, 6, 7, 8]], dtype=np.int32)
    target = np.array([[9, 6, 7, 1, 2]], dtype=np.int32)
    L = np.array([3], dtype=np.int32)
    bt = np.array([[4, 2]], dtype=np.int32)
    assert orc.verify_accept(draft, target, L, bt, 16, 0)["accept_len"][0] == 0
    out = orc.verify_accept(draft, target, L, bt, 16, 1)
    assert out["accept_len"][0] == 3 and out["bonus"][0] == 1


# ----------------------------------------------------------------------------- RoPE / norm
def test_rope_hand_values():
    # hd = 2: one pair, frequency 1: (1, 0) at position p turns into (cos p, sin p).
    out = orc.rope(np.array([1.0, 0.0]), 0.5, 10000.0)
    assert np.allclose(out, [math.cos(0.5), math.sin(0.5)], atol=1e-15)
    out = orc.rope(np.array([0.0, 1.0]), 0.5, 10000.0)
    assert np.allclose(out, [-math.sin(0.5), math.cos(0.5)], atol=1e-15)
    # hd = 4: pairs (0,2) and (1,3); the second pair turns at theta^(-1/2).
    x = np.array([1.0, 2.0, 3.0, 4.0])
    p, th = 7.0, 100.0
    a0, a1 = p * 1.0, p * th ** -0.5
    want = [1 * math.cos(a0) - 3 * math.sin(a0), 2 * math.cos(a1) - 4 * math.sin(a1),
            3 * math.cos(a0) + 1 * math.sin(a0), 4 * math.cos(a1) + 2 * math.sin(a1)]
    assert np.allclose(orc.rope(x, p, th), want, atol=1e-13)


def test_rope_invariants():
    rng = np.random.default_rng(0)
    hd = 64
    q = rng.standard_normal((5, hd))
    k = rng.standard_normal((5, hd))
    assert np.array_equal(orc.rope(q, np.zeros(5), 1e6), q)            # position 0 = identity
    r = orc.rope(q, np.arange(5) * 1000.0, 1e6)
    assert np.allclose((r ** 2).sum(-1), (q ** 2).sum(-1), rtol=1e-12)  # a rotation
    half = hd // 2
    assert np.allclose(r[:, :half] ** 2 + r[:, half:] ** 2,
                       q[:, :half] ** 2 + q[:, half:] ** 2, rtol=1e-10)
    # scores depend on the position difference only
    d1 = (orc.rope(q, np.full(5, 17.0), 1e4) * orc.rope(k, np.full(5, 5.0), 1e4)).sum(-1)
    d2 = (orc.rope(q, np.full(5, 1012.0), 1e4) * orc.rope(k, np.full(5, 1000.0), 1e4)).sum(-1)
    assert np.allclose(d1, d2, atol=1e-9)


def test_rmsnorm_closed_form():
    x = np.array([[3.0, 4.0]])
    g = np.array([2.0, 0.5])
    # mean square = 12.5
    want = g * x / math.sqrt(12.5 + 1e-6)
    assert np.allclose(orc.rmsnorm(x, g, 1e-6), want, atol=1e-15)
    y = orc.rmsnorm(np.random.default_rng(0).standard_normal((4, 256)) * 7, np.ones(256), 0.0)
    assert np.allclose((y ** 2).mean(-1), 1.0)


# ----------------------------------------------------------------------------- part 2
def _tiny(norm=True, **kw):
    wl = synth.workload("cfg1")
    wl = synth.scaled(wl, hidden_norm=norm, **kw)
    cfg = oracle_config(wl.shape)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 5))
    return wl, cfg, w


def _split_for(wl, m, seed=0):
    lay = synth.make_layout(wl, seed)
    rng = np.random.default_rng(seed + 77)
    draft, target = synth.make_tokens(wl, rng, np.asarray(m, dtype=np.int32))
    sp = orc.verify_accept(draft, target, lay["committed_len"], lay["block_table"], wl.shape.page, 0)
    assert np.array_equal(sp["accept_len"], m)
    return sp, lay


def test_project_linearity_in_carry_embedding():
    """Norm off: Phi(h + E) = Phi(h) + Phi(E) row-wise, also after the key rotation."""
    wl, cfg, w = _tiny(norm=False, S=2)
    sp, _ = _split_for(wl, [3, 0])
    H = synth.make_round(wl, 0, 0)["H"].astype(np.float64)
    J = orc.project_kv(H, sp, w, cfg, orc.MODE_CARRY)
    w0 = dict(w, e_carry=np.zeros_like(w["e_carry"]))
    J0 = orc.project_kv(H, sp, w0, cfg, orc.MODE_CARRY)
    # Phi(E) alone, at each row's own position
    HE = np.tile(w["e_carry"], (wl.R, 1))
    sp_all = dict(sp, accept_len=np.array([wl.shape.W] * wl.S))       # nothing rejected
    JE = orc.project_kv(HE, sp_all, w0, cfg, orc.MODE_CARRY)
    rej = np.repeat(sp["accept_len"], wl.shape.W) <= np.tile(np.arange(wl.shape.W), wl.S)
    assert rej.sum() == 5 + 8
    assert np.allclose(J[:, rej], J0[:, rej] + JE[:, rej], atol=1e-12)
    assert np.array_equal(J[:, ~rej], J0[:, ~rej])                  # accepted rows never see E


@pytest.mark.parametrize("norm", [False, True])
def test_rejected_rows_use_the_same_path_when_E_is_zero(norm):
    """E_carry = 0: a rejected row's K/V equal what the accepted-row path gives for it."""
    wl, cfg, w = _tiny(norm=norm, S=2)
    w0 = dict(w, e_carry=np.zeros_like(w["e_carry"]))
    H = synth.make_round(wl, 0, 1)["H"]
    sp, _ = _split_for(wl, [2, 5])
    J = orc.project_kv(H, sp, w0, cfg, orc.MODE_CARRY)
    sp_all = dict(sp, accept_len=np.array([wl.shape.W] * wl.S))
    Jb = orc.project_kv(H, sp_all, w0, cfg, orc.MODE_BASELINE)
    assert np.array_equal(J, Jb)
    # and with E != 0 the rejected rows do change, the accepted ones do not
    JE = orc.project_kv(H, sp, w, cfg, orc.MODE_CARRY)
    rej = np.repeat(sp["accept_len"], wl.shape.W) <= np.tile(np.arange(wl.shape.W), wl.S)
    assert np.array_equal(JE[:, ~rej], J[:, ~rej])
    assert np.abs(JE[:, rej] - J[:, rej]).max() > 1e-3


def test_baseline_projects_accepted_rows_only():
    wl, cfg, w = _tiny(S=2)
    H = synth.make_round(wl, 0, 2)["H"]
    sp, _ = _split_for(wl, [2, 8])
    Jb = orc.project_kv(H, sp, w, cfg, orc.MODE_BASELINE)
    Jc = orc.project_kv(H, sp, w, cfg, orc.MODE_CARRY)
    rej = np.repeat(sp["accept_len"], wl.shape.W) <= np.tile(np.arange(wl.shape.W), wl.S)
    assert np.isnan(Jb[:, rej]).all()
    assert np.array_equal(Jb[:, ~rej], Jc[:, ~rej])


def test_project_with_selection_weights_is_a_copy():
    """One-hot F, K, V (norm off) and position 0: the outputs are exact copies of H entries."""
    wl, cfg, w = _tiny(norm=False)
    D, Din, kvw = cfg.d_model, cfg.d_in, cfg.n_kv * cfg.hd
    rng = np.random.default_rng(4)
    sel_f = rng.permutation(Din)[:D]
    sel_k = rng.permutation(D)[:kvw]
    sel_v = rng.permutation(D)[:kvw]
    w = dict(w)
    w["fc"] = np.zeros((D, Din)); w["fc"][np.arange(D), sel_f] = 1.0
    w["wk"] = np.zeros((1, kvw, D)); w["wk"][0, np.arange(kvw), sel_k] = 1.0
    w["wv"] = np.zeros((1, kvw, D)); w["wv"][0, np.arange(kvw), sel_v] = 1.0
    H = synth.make_round(wl, 0, 0)["H"].astype(np.float64)
    W = cfg.W
    sp = {"accept_len": np.array([3]), "row_pos": np.zeros(W, dtype=np.int32)}
    J = orc.project_kv(H, sp, w, cfg, orc.MODE_CARRY)
    Hk = H.copy(); Hk[3:] += w["e_carry"]
    assert np.array_equal(J[0, :, 1].reshape(W, kvw), Hk[:, sel_f][:, sel_v])
    assert np.array_equal(J[0, :, 0].reshape(W, kvw), Hk[:, sel_f][:, sel_k])


def test_project_against_torch_linear():
    """The same maps through torch's float64 linear layers and an explicit rotation."""
    wl, cfg, w = _tiny(S=2)
    H = synth.make_round(wl, 0, 3)["H"]
    sp, _ = _split_for(wl, [4, 1])
    J = orc.project_kv(H, sp, w, cfg, orc.MODE_CARRY)
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    Ht = t(H).clone()
    for s, m in enumerate([4, 1]):
        Ht[s * 8 + m:(s + 1) * 8] += t(w["e_carry"])
    Z = torch.nn.functional.linear(Ht, t(w["fc"]))
    Z = Z * torch.rsqrt((Z * Z).mean(-1, keepdim=True) + cfg.rms_eps) * t(w["g_hidden"])
    K = torch.nn.functional.linear(Z, t(w["wk"][0])).reshape(-1, cfg.n_kv, cfg.hd)
    V = torch.nn.functional.linear(Z, t(w["wv"][0])).reshape(-1, cfg.n_kv, cfg.hd)
    half = cfg.hd // 2
    inv = cfg.rope_theta ** (-torch.arange(half, dtype=torch.float64) * 2 / cfg.hd)
    ang = t(sp["row_pos"])[:, None, None] * inv
    Kr = torch.cat([K[..., :half] * ang.cos() - K[..., half:] * ang.sin(),
                    K[..., half:] * ang.cos() + K[..., :half] * ang.sin()], -1)
    assert np.allclose(J[0, :, 0], Kr.numpy(), atol=1e-12)
    assert np.allclose(J[0, :, 1], V.numpy(), atol=1e-12)


# ----------------------------------------------------------------------------- part 3
def test_scatter_semantics_over_rounds():
    """Carry never exceeds W rows, is replaced each round, starts empty; rejected rows never
    reach the committed cache; committed rows are exact copies and older rows never change."""
    wl = synth.scaled(synth.workload("cfg1"), S=3, ctx=(5, 40), n_rounds=6)
    cfg, st, lay = oracle_state(wl, 2)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 2))
    assert (st.carry_len == 0).all() and np.isnan(st.carry).all()
    W, page = cfg.W, cfg.page
    for r in range(6):
        rd = synth.make_round(wl, 2, r)
        pool_before = st.pool.copy()
        L0 = st.committed_len.copy()
        sp = orc.verify_accept(rd["draft"], rd["target"], st.committed_len, st.block_table, page, wl.n_forced)
        J = orc.project_kv(rd["H"], sp, w, cfg, orc.MODE_CARRY)
        orc.scatter_kv(J, sp, st, orc.MODE_CARRY)
        m = sp["accept_len"]
        assert np.array_equal(st.committed_len, L0 + m)
        assert np.array_equal(st.carry_len, W - m) and (st.carry_len <= W).all()
        changed = np.zeros(st.pool.shape, dtype=bool)
        for s in range(wl.S):
            c = int(st.carry_len[s])
            assert np.isnan(st.carry[:, s, :, :, c:, :]).all()          # old carry is gone
            for p in range(W):
                pos = int(L0[s]) + p
                pg, off = st.block_table[s, pos // page], pos % page
                if p < m[s]:
                    assert np.array_equal(st.pool[:, pg, :, :, off, :],
                                          np.transpose(J[:, s * W + p], (0, 2, 1, 3)))
                    changed[:, pg, :, :, off, :] = True
                else:
                    assert np.array_equal(st.carry[:, s, :, :, p - m[s], :],
                                          np.transpose(J[:, s * W + p], (0, 2, 1, 3)))
        assert np.array_equal(st.pool[~changed], pool_before[~changed])


def test_baseline_scatter_leaves_carry_empty():
    wl = synth.scaled(synth.workload("cfg1"), S=2, ctx=(5, 40))
    cfg, st, _ = oracle_state(wl, 2)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 2))
    rd = synth.make_round(wl, 2, 0)
    orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, wl.n_forced, orc.MODE_BASELINE)
    assert (st.carry_len == 0).all() and np.isnan(st.carry).all()


# ----------------------------------------------------------------------------- part 4
def _attn_case(seed=0, S=2, carry=True):
    wl = synth.scaled(synth.workload("cfg1"), S=S, ctx=(3, 45))
    cfg, st, lay = oracle_state(wl, seed)
    rng = np.random.default_rng(seed + 10)
    if carry:
        st.carry_len[:] = rng.integers(1, cfg.W + 1, size=S)
        for s in range(S):
            c = int(st.carry_len[s])
            st.carry[:, s, :, :, :c, :] = rng.standard_normal((cfg.n_layers, cfg.n_kv, 2, c, cfg.hd))
    q = rng.standard_normal((S, cfg.W, cfg.n_q, cfg.hd))
    kb = rng.standard_normal((S, cfg.W, cfg.n_kv, cfg.hd))
    vb = rng.standard_normal((S, cfg.W, cfg.n_kv, cfg.hd))
    return wl, cfg, st, q, kb, vb


def _rope_scalar(x, pos, theta):
    """Independent scalar-loop rotation used by the brute-force attention."""
    hd = len(x)
    half = hd // 2
    out = [0.0] * hd
    for j in range(half):
        a = pos * theta ** (-2.0 * j / hd)
        out[j] = x[j] * math.cos(a) - x[j + half] * math.sin(a)
        out[j + half] = x[j + half] * math.cos(a) + x[j] * math.sin(a)
    return out


def test_attention_brute_force_loops():
    """Materialised scores in pure Python loops with a page-table walk of its own."""
    wl, cfg, st, q, kb, vb = _attn_case(seed=1, S=2)
    out, mass = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    rep = cfg.n_q // cfg.n_kv
    for s in range(2):
        L, c = int(st.committed_len[s]), int(st.carry_len[s])
        for i in (0, cfg.W - 1):
            for g in (0, cfg.n_q - 1):
                h = g // rep
                qq = _rope_scalar(list(q[s, i, g]), L + i, cfg.rope_theta)
                keys, vals = [], []
                for t in range(L):
                    pg = int(st.block_table[s, t // cfg.page])
                    keys.append(list(st.pool[0, pg, h, 0, t % cfg.page]))
                    vals.append(list(st.pool[0, pg, h, 1, t % cfg.page]))
                for u in range(c):
                    keys.append(list(st.carry[0, s, h, 0, u]))
                    vals.append(list(st.carry[0, s, h, 1, u]))
                for jb in range(cfg.W):
                    keys.append(_rope_scalar(list(kb[s, jb, h]), L + jb, cfg.rope_theta))
                    vals.append(list(vb[s, jb, h]))
                sc = [sum(a * b for a, b in zip(qq, k)) / math.sqrt(cfg.hd) for k in keys]
                mx = max(sc)
                e = [math.exp(v - mx) for v in sc]
                z = sum(e)
                o = [sum(e[t] * vals[t][d] for t in range(len(e))) / z for d in range(cfg.hd)]
                assert np.allclose(out[s, i, g], o, atol=1e-12)
                assert abs(mass[s, i, g] - sum(e[L:L + c]) / z) < 1e-12


def test_attention_is_plain_sdpa_over_concatenated_keys():
    """Once [C; U; block] is concatenated and GQA heads repeated, it is library SDPA."""
    wl, cfg, st, q, kb, vb = _attn_case(seed=2, S=2)
    out, _ = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    rep = cfg.n_q // cfg.n_kv
    for s in range(2):
        L, c = int(st.committed_len[s]), int(st.carry_len[s])
        pos = L + np.arange(cfg.W)
        t_idx = np.arange(L)
        pg = st.block_table[s, t_idx // cfg.page]
        Kc = np.stack([st.pool[0, pg[t], :, 0, t % cfg.page] for t in range(L)], 0)    # [L, n_kv, hd]
        Vc = np.stack([st.pool[0, pg[t], :, 1, t % cfg.page] for t in range(L)], 0)
        Ku = np.transpose(st.carry[0, s, :, 0, :c], (1, 0, 2))
        Vu = np.transpose(st.carry[0, s, :, 1, :c], (1, 0, 2))
        Kb = np.stack([[_rope_scalar(list(kb[s, j, h]), int(pos[j]), cfg.rope_theta)
                        for h in range(cfg.n_kv)] for j in range(cfg.W)], 0)
        K = np.concatenate([Kc, Ku, Kb], 0)
        V = np.concatenate([Vc, Vu, vb[s]], 0)
        Q = np.stack([[_rope_scalar(list(q[s, i, g]), int(pos[i]), cfg.rope_theta)
                       for g in range(cfg.n_q)] for i in range(cfg.W)], 0)
        Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(rep, 0)   # [n_q, T, hd]
        Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(rep, 0)
        Qt = torch.from_numpy(Q).permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt)      # [n_q, W, hd]
        assert np.allclose(out[s], ref.permute(1, 0, 2).numpy(), atol=1e-11)


def test_attention_closed_forms():
    wl = synth.scaled(synth.workload("cfg1"), S=1, ctx=(0, 0), W=1)
    cfg, st, _ = oracle_state(wl, 0)
    rng = np.random.default_rng(0)
    # one key in total (the block row itself): output = its V
    q = rng.standard_normal((1, 1, cfg.n_q, cfg.hd))
    kb = rng.standard_normal((1, 1, cfg.n_kv, cfg.hd))
    vb = rng.standard_normal((1, 1, cfg.n_kv, cfg.hd))
    out, _ = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    rep = cfg.n_q // cfg.n_kv
    for g in range(cfg.n_q):
        assert np.allclose(out[0, 0, g], vb[0, 0, g // rep], atol=1e-15)
    # identical keys everywhere: output = mean of the values
    wl = synth.scaled(synth.workload("cfg1"), S=1, ctx=(20, 20))
    cfg, st, _ = oracle_state(wl, 0)
    st.pool[:, :, :, 0] = 0.0                                    # all committed keys = 0
    kb = np.zeros((1, cfg.W, cfg.n_kv, cfg.hd))                  # rotation of 0 is 0
    vb = rng.standard_normal((1, cfg.W, cfg.n_kv, cfg.hd))
    q = rng.standard_normal((1, cfg.W, cfg.n_q, cfg.hd))
    out, _ = orc.block_attn(0, q, kb, vb, st, use_carry=False)
    pg = st.block_table[0, np.arange(20) // cfg.page]
    for g in range(cfg.n_q):
        h = g // rep
        vals = [st.pool[0, pg[t], h, 1, t % cfg.page] for t in range(20)] + list(vb[0, :, h])
        assert np.allclose(out[0, 3, g], np.mean(vals, axis=0), atol=1e-13)
    # two keys with scores 0 and ln 3 (hd = 4, scale 1/2): weights 1/4 and 3/4
    wl = synth.scaled(synth.workload("cfg1"), S=1, ctx=(1, 1), W=1, hd=4, n_q=1, n_kv=1, d_model=4)
    cfg, st, _ = oracle_state(wl, 0)
    pg = st.block_table[0, 0]
    st.pool[0, pg, 0, 0, 0] = [0.0, 0.0, 0.0, 0.0]
    st.pool[0, pg, 0, 1, 0] = [1.0, 0.0, 0.0, 0.0]
    q = np.array([[[[2 * math.log(3.0), 0.0, 0.0, 0.0]]]])
    kb = np.array([[[[1.0, 0.0, 0.0, 0.0]]]])
    vb = np.array([[[[0.0, 1.0, 0.0, 0.0]]]])
    # q and k_blk sit at the same position, so the rotation leaves their product unchanged
    out, _ = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    golden = os.path.join(os.path.dirname(__file__), "golden", "attention_two_keys.txt")
    want = np.loadtxt(golden, comments="#")
    assert want.shape == (4,) and np.allclose(out[0, 0, 0], want, atol=1e-14)


def test_attention_masked_carry_equals_baseline_and_mass():
    wl, cfg, st, q, kb, vb = _attn_case(seed=3)
    out_c, mass_c = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    out_b, mass_b = orc.block_attn(0, q, kb, vb, st, use_carry=False)
    assert np.abs(out_c - out_b).max() > 1e-3 and (mass_c > 0).all() and (mass_c < 1).all()
    assert (mass_b == 0).all()
    keep = st.carry_len.copy()
    st.carry_len[:] = 0                                            # empty carry = baseline
    out_0, _ = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    assert np.array_equal(out_0, out_b)
    st.carry_len[:] = keep


def test_attention_page_permutation_invariance():
    wl, cfg, st, q, kb, vb = _attn_case(seed=4)
    out, _ = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    n_pages = st.pool.shape[1]
    perm = np.random.default_rng(9).permutation(n_pages)
    inv = np.argsort(perm)
    st2 = orc.OracleState(cfg, st.S, n_pages, perm[st.block_table], st.committed_len)
    st2.pool = st.pool[:, inv]
    st2.carry, st2.carry_len = st.carry, st.carry_len
    out2, _ = orc.block_attn(0, q, kb, vb, st2, use_carry=True)
    assert np.array_equal(out, out2)


def test_attention_depends_on_relative_position_only():
    """Move every row (committed, carried, block) delta positions later, re-rotating the stored
    keys by delta: the outputs must not change.  The delta vacated leading positions hold
    zero keys / zero values, whose scores are 0 whatever the rotation; the expected result is
    computed directly with those filler rows in front."""
    wl, cfg, st, q, kb, vb = _attn_case(seed=4)
    delta = 37
    n_pages = st.pool.shape[1]
    bt = np.zeros((st.S, 16), dtype=np.int64)
    shifted = orc.OracleState(cfg, st.S, n_pages + 64, bt, st.committed_len + delta)
    stale = orc.OracleState(cfg, st.S, n_pages + 64, bt, st.committed_len + delta)
    nxt = 0
    for s in range(st.S):
        L = int(st.committed_len[s])
        npg = (L + delta + cfg.page - 1) // cfg.page
        bt[s, :npg] = np.arange(nxt, nxt + npg); nxt += npg
        shifted.block_table[s] = bt[s]; stale.block_table[s] = bt[s]
        K, V, c = orc.gather_ctx(st, 0, s, True)                   # [n_kv, L + c, hd]
        Kr = orc.rope(K, np.full(K.shape[1], float(delta))[None, :], cfg.rope_theta)
        for dst, Kuse in ((shifted, Kr), (stale, K)):
            for t in range(L):
                pos = t + delta
                pg = dst.block_table[s, pos // cfg.page]
                dst.pool[0, pg, :, 0, pos % cfg.page] = Kuse[:, t]
                dst.pool[0, pg, :, 1, pos % cfg.page] = V[:, t]
            dst.carry[0, s, :, 0, :c] = Kuse[:, L:L + c]
            dst.carry[0, s, :, 1, :c] = V[:, L:L + c]
            dst.carry_len[s] = c
    out_shift, _ = orc.block_attn(0, q, kb, vb, shifted, use_carry=True)
    out_stale, _ = orc.block_attn(0, q, kb, vb, stale, use_carry=True)
    assert np.abs(out_stale - out_shift).max() > 1e-4              # keys do carry their position
    rep = cfg.n_q // cfg.n_kv
    for s in range(st.S):
        L = int(st.committed_len[s])
        K, V, c = orc.gather_ctx(st, 0, s, True)
        pos = (L + np.arange(cfg.W)).astype(np.float64)
        qr = orc.rope(q[s], pos[:, None], cfg.rope_theta)
        kr = orc.rope(kb[s], pos[:, None], cfg.rope_theta)
        for g in range(cfg.n_q):
            h = g // rep
            Kall = np.concatenate([np.zeros((delta, cfg.hd)), K[h], kr[:, h]], 0)
            Vall = np.concatenate([np.zeros((delta, cfg.hd)), V[h], vb[s][:, h]], 0)
            sc = qr[:, g] @ Kall.T / math.sqrt(cfg.hd)
            pr = np.exp(sc - sc.max(1, keepdims=True)); pr /= pr.sum(1, keepdims=True)
            assert np.allclose(out_shift[s, :, g], pr @ Vall, atol=1e-9)


# ----------------------------------------------------------------------------- part 5
def test_lm_head_planted_maximum_and_ties():
    wl, cfg, w = _tiny()
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6, cfg.d_model))
    y = orc.rmsnorm(x, w["g_final"], cfg.rms_eps)
    for row, v in enumerate([0, 127, 128, 500, cfg.vocab - 2, cfg.vocab - 1]):
        w2 = dict(w); emb = w["emb"].copy(); emb[v] = y[row] * 10.0; w2["emb"] = emb
        tok, gap, _ = orc.lm_head_argmax(x, w2, cfg)
        assert tok[row] == v and gap[row] > 0
    # exact tie between two vocabulary rows: the lower id wins, the gap is zero
    w2 = dict(w); emb = w["emb"].copy(); emb[700] = y[2] * 10.0; emb[33] = emb[700]; w2["emb"] = emb
    tok, gap, _ = orc.lm_head_argmax(x, w2, cfg)
    assert tok[2] == 33 and gap[2] == 0.0


def test_lm_head_brute_force():
    wl, cfg, w = _tiny()
    x = np.random.default_rng(1).standard_normal((3, cfg.d_model))
    tok, gap, _ = orc.lm_head_argmax(x, w, cfg)
    for r in range(3):
        ms = math.sqrt(sum(v * v for v in x[r]) / cfg.d_model + cfg.rms_eps)
        y = [w["g_final"][d] * x[r, d] / ms for d in range(cfg.d_model)]
        logits = [math.fsum(w["emb"][v, d] * y[d] for d in range(cfg.d_model)) for v in range(cfg.vocab)]
        best = max(range(cfg.vocab), key=lambda v: (logits[v], -v))
        srt = sorted(logits)
        assert tok[r] == best
        assert abs(gap[r] - (srt[-1] - srt[-2])) < 1e-12


# ----------------------------------------------------------------------------- whole round
def test_full_acceptance_round_equals_baseline_round():
    """Full acceptance leaves U empty, so the round is the no-carryover drafter's round."""
    wl = synth.scaled(synth.workload("cfg1"), S=2, ctx=(20, 60), accept=("fixed_m", 8), n_forced=0)
    cfg, st_c, _ = oracle_state(wl, 1)
    _, st_b, _ = oracle_state(wl, 1)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 1))
    w["wo"] = w["wo"] * 40.0                                       # make the attention path matter
    for r in range(3):
        rd = synth.make_round(wl, 1, r)
        rc = orc.draft_round(rd["draft"], rd["target"], rd["H"], st_c, w, 0, orc.MODE_CARRY, keep_logits=True)
        rb = orc.draft_round(rd["draft"], rd["target"], rd["H"], st_b, w, 0, orc.MODE_BASELINE, keep_logits=True)
        assert (st_c.carry_len == 0).all()
        assert np.array_equal(rc["logits"], rb["logits"])
        assert np.array_equal(rc["next_draft"], rb["next_draft"])
        assert np.array_equal(st_c.pool, st_b.pool)


def test_partial_acceptance_differs_from_baseline_and_commits_the_same():
    wl = synth.scaled(synth.workload("cfg1"), S=2, ctx=(20, 60))
    cfg, st_c, _ = oracle_state(wl, 1)
    _, st_b, _ = oracle_state(wl, 1)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 1))
    w["wo"] = w["wo"] * 40.0
    differs = False
    for r in range(4):
        rd = synth.make_round(wl, 1, r)
        rc = orc.draft_round(rd["draft"], rd["target"], rd["H"], st_c, w, 1, orc.MODE_CARRY)
        rb = orc.draft_round(rd["draft"], rd["target"], rd["H"], st_b, w, 1, orc.MODE_BASELINE)
        # the acceptance rule and the committed cache do not depend on carryover
        assert np.array_equal(rc["split"]["accept_len"], rb["split"]["accept_len"])
        assert np.array_equal(st_c.pool, st_b.pool)
        assert np.array_equal(st_c.committed_len, st_b.committed_len)
        differs |= np.abs(rc["x_final"] - rb["x_final"]).max() > 1e-6
    assert differs


def test_committed_cache_equals_from_scratch_recomputation():
    """After many rounds the committed rows are exactly Phi of the concatenated accepted
    hiddens at positions 0.., computed in one go without any paging."""
    wl = synth.scaled(synth.workload("cfg1"), S=2, ctx=(0, 0), n_rounds=16)
    cfg, st, _ = oracle_state(wl, 6, fill_pool=False)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 6))
    kept = [[], []]
    for r in range(16):
        rd = synth.make_round(wl, 6, r)
        res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
        for s in range(2):
            kept[s].append(rd["H"][s * cfg.W: s * cfg.W + int(rd["m"][s])])
    for s in range(2):
        Hs = np.concatenate(kept[s], 0).astype(np.float64)
        L = Hs.shape[0]
        assert L == st.committed_len[s]
        Z = Hs @ w["fc"].T
        Z = w["g_hidden"] * Z / np.sqrt((Z * Z).mean(-1, keepdims=True) + cfg.rms_eps)
        K = orc.rope((Z @ w["wk"][0].T).reshape(L, cfg.n_kv, cfg.hd), np.arange(L)[:, None], cfg.rope_theta)
        V = (Z @ w["wv"][0].T).reshape(L, cfg.n_kv, cfg.hd)
        Kc, Vc, _ = orc.gather_ctx(st, 0, s, use_carry=False)
        assert np.allclose(np.transpose(Kc, (1, 0, 2)), K, atol=1e-12)
        assert np.allclose(np.transpose(Vc, (1, 0, 2)), V, atol=1e-12)


def test_round_is_deterministic_and_next_draft_shape():
    wl = small_bf16()
    outs = []
    for _ in range(2):
        cfg, st, _ = oracle_state(wl, 0)
        w = orc.prepare_weights(synth.make_weights(wl.shape, 0))
        rd = synth.make_round(wl, 0, 0)
        res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
        outs.append(res)
    assert np.array_equal(outs[0]["x_final"], outs[1]["x_final"])
    nd = outs[0]["next_draft"]
    assert nd.shape == (wl.S, wl.shape.W) and np.array_equal(nd[:, 0], outs[0]["split"]["bonus"])
    assert np.array_equal(nd[:, 1:], outs[0]["tok"][:, 1:])


# ----------------------------------------------------------------------------- the drafter pass: attention sub-layer
def _body_case(n_layers, seed=9, S=2):
    """A tiny drafter (D = 32) after one carry-mode round, so C_l, U_l and the bonus tokens are real;
    the attention matrices are scaled up so the sub-layer moves the residual stream by O(1)."""
    wl = synth.scaled(synth.workload("cfg1"), S=S, ctx=(5, 30), n_layers=n_layers, d_target=16, n_cap=2,
                      d_model=32, n_q=4, n_kv=2, hd=8, vocab=64, W=4, n_rounds=2,
                      accept=("rej_uniform", 1, 3))
    cfg, st, _ = oracle_state(wl, seed)
    w = orc.prepare_weights(synth.make_weights(wl.shape, seed))
    for k in ("wq", "wk", "wv", "wo"):
        w[k] = w[k] * 12.0
    rd = synth.make_round(wl, seed, 0)
    res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY, keep_logits=True)
    assert st.carry_len.max() > 0                              # carried rows are part of what is read
    return wl, cfg, st, w, res


def _matvec_loops(Wm, v):
    """y_i = sum_k W[i, k] v[k] for a matrix stored [out, in], written out."""
    return [sum(float(Wm[i, k]) * v[k] for k in range(Wm.shape[1])) for i in range(Wm.shape[0])]


def _rms_gain_loops(x, g, eps):
    ms = sum(v * v for v in x) / len(x)
    return [float(g[k]) * x[k] / math.sqrt(ms + eps) for k in range(len(x))]


def test_draft_block_one_layer_written_out_by_hand():
    """One drafter layer, no MLP: for every block row a = g_attn * x0 / rms(x0); q, k_b, v_b = W a with explicit
    sums; the (separately pinned) block attention on them; x1 = x0 + W_o o; y = g_final * x1 / rms(x1);
    token = first index of the largest Emb[v] . y."""
    wl, cfg, st, w, res = _body_case(n_layers=1)
    S, W, D = wl.S, cfg.W, cfg.d_model
    bonus = res["split"]["bonus"]
    x0 = []
    for s in range(S):
        for i in range(W):
            t = int(bonus[s]) if i == 0 else cfg.mask_token_id
            x0.append([float(v) for v in w["emb"][t]])
    q = np.zeros((S, W, cfg.n_q, cfg.hd)); kb = np.zeros((S, W, cfg.n_kv, cfg.hd)); vb = np.zeros_like(kb)
    for r in range(S * W):
        a = _rms_gain_loops(x0[r], w["g_attn"][0], cfg.rms_eps)
        q[r // W, r % W] = np.array(_matvec_loops(w["wq"][0], a)).reshape(cfg.n_q, cfg.hd)
        kb[r // W, r % W] = np.array(_matvec_loops(w["wk"][0], a)).reshape(cfg.n_kv, cfg.hd)
        vb[r // W, r % W] = np.array(_matvec_loops(w["wv"][0], a)).reshape(cfg.n_kv, cfg.hd)
    o, _ = orc.block_attn(0, q, kb, vb, st, use_carry=True)
    o = o.reshape(S * W, cfg.n_q * cfg.hd)
    assert np.allclose(res["attn_out"][0], o, atol=1e-10)
    for r in range(S * W):
        wo_o = _matvec_loops(w["wo"][0], [float(v) for v in o[r]])
        x1 = [x0[r][i] + wo_o[i] for i in range(D)]
        assert np.allclose(res["x_final"][r], x1, atol=1e-10)
        assert max(abs(v) for v in wo_o) > 1e-2                # the branch under test is not negligible
        y = _rms_gain_loops(x1, w["g_final"], cfg.rms_eps)
        logits = [sum(float(w["emb"][v, k]) * y[k] for k in range(D)) for v in range(cfg.vocab)]
        assert np.allclose(res["logits"][r], logits, atol=1e-10)
        assert int(res["tok"].reshape(-1)[r]) == logits.index(max(logits))


def _torch_body(cfg, st, w, bonus, S, *, gains=None, wo_of=None, order=None, norm_input=True, residual=True):
    """The attention-only drafter body through torch float64 linear / rms_norm, the oracle's own block
    attention as the (pinned) inner step.  The keyword switches build the plausible mistakes."""
    F = torch.nn.functional
    W = cfg.W
    toks = np.full((S, W), cfg.mask_token_id, dtype=np.int64)
    toks[:, 0] = bonus
    x = torch.from_numpy(w["emb"])[torch.from_numpy(toks.reshape(-1))]
    gains = w["g_attn"] if gains is None else gains
    outs = []
    for l in (range(cfg.n_layers) if order is None else order):
        a = F.rms_norm(x, (cfg.d_model,), torch.from_numpy(np.ascontiguousarray(gains[l])), cfg.rms_eps)
        if not norm_input:
            a = x
        q = F.linear(a, torch.from_numpy(w["wq"][l])).numpy().reshape(S, W, cfg.n_q, cfg.hd)
        kb = F.linear(a, torch.from_numpy(w["wk"][l])).numpy().reshape(S, W, cfg.n_kv, cfg.hd)
        vb = F.linear(a, torch.from_numpy(w["wv"][l])).numpy().reshape(S, W, cfg.n_kv, cfg.hd)
        o, _ = orc.block_attn(l, q, kb, vb, st, use_carry=True)
        o = torch.from_numpy(o.reshape(S * W, -1))
        outs.append(o.numpy())
        wo = w["wo"][l] if wo_of is None else wo_of(w["wo"][l])
        upd = F.linear(o, torch.from_numpy(np.ascontiguousarray(wo)))
        x = x + upd if residual else upd
    return x.numpy(), outs


def test_draft_block_two_layers_against_torch_ops():
    """Two layers: layer order, g_attn indexed by layer, the residual carried from layer to layer."""
    wl, cfg, st, w, res = _body_case(n_layers=2, seed=11)
    x, outs = _torch_body(cfg, st, w, res["split"]["bonus"], wl.S)
    assert np.allclose(res["x_final"], x, atol=1e-11)
    for l in range(2):
        assert np.allclose(res["attn_out"][l], outs[l], atol=1e-11)
    y = torch.nn.functional.rms_norm(torch.from_numpy(x), (cfg.d_model,), torch.from_numpy(w["g_final"]), cfg.rms_eps)
    logits = torch.nn.functional.linear(y, torch.from_numpy(w["emb"])).numpy()
    assert np.allclose(res["logits"], logits, atol=1e-11)
    assert np.array_equal(res["tok"].reshape(-1), logits.argmax(1))


def test_draft_block_pins_would_catch_the_plausible_mistakes():
    """Each mistake a reader might make in the body changes x_final by far more than the pins' tolerance,
    so the two tests above do tell them apart from the right computation."""
    wl, cfg, st, w, res = _body_case(n_layers=2, seed=11)
    bonus, S = res["split"]["bonus"], wl.S
    good = res["x_final"]
    wrong = {
        "gains of the two layers swapped": dict(gains=w["g_attn"][::-1]),
        "no gain": dict(gains=np.ones_like(w["g_attn"])),
        "final gain in place of the layer's": dict(gains=np.stack([w["g_final"]] * 2)),
        "W_o transposed": dict(wo_of=lambda m: m.T),
        "q/k/v from the un-normalised stream": dict(norm_input=False),
        "residual dropped": dict(residual=False),
        "layers in the wrong order": dict(order=[1, 0]),
    }
    for what, kw in wrong.items():
        x, _ = _torch_body(cfg, st, w, bonus, S, **kw)
        assert np.abs(x - good).max() > 1e-3, what
    # the embedding of the block: bonus in row 0, MASK elsewhere
    x, _ = _torch_body(cfg, st, w, (bonus + 1) % cfg.vocab, S)
    assert np.abs(x - good).max() > 1e-3


# ----------------------------------------------------------------------------- the complete layer
def _full_layer_workload(**kw):
    args = dict(S=2, ctx=(20, 60), d_ff=96, qk_norm=True, n_layers=2, n_rounds=4)
    args.update(kw)
    return synth.scaled(synth.workload("cfg1"), **args)


def test_silu_closed_form():
    x = np.array([0.0, 1.0, -1.0, 30.0, -30.0, math.log(3.0)])
    got = orc.silu(x)
    exp = [0.0, 1.0 / (1.0 + math.exp(-1.0)), -1.0 / (1.0 + math.e), 30.0, 0.0, math.log(3.0) * 0.75]
    assert np.allclose(got, exp, atol=1e-11)
    # silu(x) - silu(-x) = x  (sigmoid(x) + sigmoid(-x) = 1)
    y = np.linspace(-6, 6, 41)
    assert np.allclose(orc.silu(y) - orc.silu(-y), y, atol=1e-12)


def test_gated_mlp_against_torch_and_loops():
    rng = np.random.default_rng(3)
    b = rng.standard_normal((5, 12)); wg = rng.standard_normal((7, 12)); wu = rng.standard_normal((7, 12))
    wd = rng.standard_normal((12, 7))
    got = orc.gated_mlp(b, wg, wu, wd)
    F = torch.nn.functional
    tb, tg, tu, td = (torch.from_numpy(a) for a in (b, wg, wu, wd))
    ref = F.linear(F.silu(F.linear(tb, tg)) * F.linear(tb, tu), td).numpy()
    assert np.allclose(got, ref, atol=1e-12)
    # and element by element: a transposed operand or a swapped gate/up would show here
    for r in range(5):
        h = [sum(b[r, k] * wg[j, k] for k in range(12)) for j in range(7)]
        u = [sum(b[r, k] * wu[j, k] for k in range(12)) for j in range(7)]
        act = [hj / (1.0 + math.exp(-hj)) * uj for hj, uj in zip(h, u)]
        for i in range(12):
            assert abs(got[r, i] - sum(act[j] * wd[i, j] for j in range(7))) < 1e-10


@pytest.mark.parametrize("zeroed", ["w_down", "w_gate", "w_up"])
def test_mlp_with_a_zero_factor_is_the_attention_only_layer(zeroed):
    """silu(0) = 0, so a zero gate, a zero up-projection or a zero down-projection removes the MLP."""
    wl = _full_layer_workload(qk_norm=False)
    wl0 = synth.scaled(wl, d_ff=0)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 2))
    w[zeroed] = np.zeros_like(w[zeroed])
    w0 = {k: v for k, v in w.items() if k not in ("w_gate", "w_up", "w_down", "g_mlp")}
    _, st, _ = oracle_state(wl, 2)
    _, st0, _ = oracle_state(wl0, 2)
    for r in range(2):
        rd = synth.make_round(wl, 2, r)
        a = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
        b = orc.draft_round(rd["draft"], rd["target"], rd["H"], st0, w0, 1, orc.MODE_CARRY)
        assert np.array_equal(a["x_final"], b["x_final"]) and np.array_equal(a["tok"], b["tok"])


def test_mlp_residual_written_out_for_one_layer():
    """One layer with W_o = 0: x_final = x0 + MLP(N(x0) g_mlp), x0 the embedded block."""
    wl = _full_layer_workload(n_layers=1, qk_norm=False, S=1)
    cfg, st, _ = oracle_state(wl, 4)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 4))
    w["wo"] = np.zeros_like(w["wo"])
    for k in ("w_gate", "w_up", "w_down"):
        w[k] = w[k] * 25.0                                   # make the MLP term large enough to matter
    rd = synth.make_round(wl, 4, 0)
    res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
    toks = [int(res["split"]["bonus"][0])] + [cfg.mask_token_id] * (cfg.W - 1)
    for i, t in enumerate(toks):
        x0 = w["emb"][t]
        b = w["g_mlp"][0] * x0 / math.sqrt(float(np.mean(x0 * x0)) + cfg.rms_eps)
        g = w["w_gate"][0] @ b
        u = w["w_up"][0] @ b
        want = x0 + w["w_down"][0] @ (g / (1.0 + np.exp(-g)) * u)
        assert np.allclose(res["x_final"][i], want, atol=1e-10)
        assert np.abs(want - x0).max() > 1e-3


def test_qk_norm_makes_unit_mean_square_keys_and_ignores_projection_scale():
    wl = _full_layer_workload(d_ff=0, rms_eps=0.0)
    cfg, st, _ = oracle_state(wl, 5)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 5))
    w["wo"] = w["wo"] * 40.0
    rd = synth.make_round(wl, 5, 0)
    res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
    # the rotation keeps a head's length, so with unit gains every cached key has mean square exactly 1
    w1 = dict(w); w1["g_knorm"] = np.ones_like(w["g_knorm"]); w1["g_qnorm"] = np.ones_like(w["g_qnorm"])
    _, st1, _ = oracle_state(wl, 5)
    res1 = orc.draft_round(rd["draft"], rd["target"], rd["H"], st1, w1, 1, orc.MODE_CARRY)
    ms = np.mean(res1["J"][:, :, 0] ** 2, axis=-1)
    assert np.allclose(ms, 1.0, atol=1e-12)
    # values are not normalised
    assert np.abs(np.mean(res1["J"][:, :, 1] ** 2, axis=-1) - 1.0).min() > 1e-3
    # a rescaled W_q or W_k changes nothing (eps = 0): queries, cached keys and block keys are all normalised
    w2 = dict(w); w2["wq"] = w["wq"] * 7.0; w2["wk"] = w["wk"] * 0.25
    _, st2, _ = oracle_state(wl, 5)
    res2 = orc.draft_round(rd["draft"], rd["target"], rd["H"], st2, w2, 1, orc.MODE_CARRY)
    assert np.allclose(res2["x_final"], res["x_final"], rtol=0, atol=1e-11)
    assert np.allclose(st2.pool, st.pool, atol=1e-12)
    # ... and without the norms the same rescaling does change the result
    wl_off = synth.scaled(wl, qk_norm=False)
    _, sa, _ = oracle_state(wl_off, 5)
    _, sb, _ = oracle_state(wl_off, 5)
    ra = orc.draft_round(rd["draft"], rd["target"], rd["H"], sa, w, 1, orc.MODE_CARRY)
    rb = orc.draft_round(rd["draft"], rd["target"], rd["H"], sb, w2, 1, orc.MODE_CARRY)
    assert np.abs(ra["x_final"] - rb["x_final"]).max() > 1e-6


def test_qk_norm_is_applied_before_the_rotation():
    """N(RoPE(k)) = RoPE(N(k)) only for a uniform gain; with a non-uniform gain the order shows.
    The cached key must equal RoPE(g * k / rms(k)) computed by hand."""
    wl = _full_layer_workload(d_ff=0, n_layers=1, S=1)
    cfg, st, _ = oracle_state(wl, 7)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 7))
    rd = synth.make_round(wl, 7, 0)
    res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
    Z = orc.fuse_features(rd["H"], np.repeat(np.arange(cfg.W)[None] >= res["split"]["accept_len"][:, None], 1, 0).reshape(-1), w, cfg)
    row = 0
    pos = int(res["split"]["row_pos"][row])
    k = (w["wk"][0] @ Z[row]).reshape(cfg.n_kv, cfg.hd)
    half = cfg.hd // 2
    for h in range(cfg.n_kv):
        kn = w["g_knorm"][0] * k[h] / math.sqrt(float(np.mean(k[h] ** 2)) + cfg.rms_eps)
        for j in range(half):
            ang = pos * cfg.rope_theta ** (-2.0 * j / cfg.hd)
            want1 = kn[j] * math.cos(ang) - kn[j + half] * math.sin(ang)
            want2 = kn[j + half] * math.cos(ang) + kn[j] * math.sin(ang)
            assert abs(res["J"][0, row, 0, h, j] - want1) < 1e-10
            assert abs(res["J"][0, row, 0, h, j + half] - want2) < 1e-10


# ----------------------------------------------------------------------------- analysis aids
def test_reconvergence_hand_examples():
    z = np.array([[5, 6, 7, 8], [5, 6, 7, 8], [5, 6, 7, 8], [1, 1, 1, 1], [5, 6, 7, 8]])
    y = np.array([[5, 6, 7, 8],      # identical: every position matches at d = 0
                  [6, 7, 8, 9],      # continuation shifted by one (a deleted token): q = 0, 1, 2 match at d = +1
                  [4, 5, 6, 7],      # shifted the other way (an inserted token): q = 1, 2, 3 match at d = -1
                  [2, 2, 2, 2],      # nothing in common
                  [7, 7, 7, 7]])     # z_2 = 7 is within one position of q = 1, 2, 3 only
    L = np.array([4, 4, 4, 4, 4])
    assert orc.reconvergence_count(z, y, L).tolist() == [4, 3, 3, 0, 3]
    # the suffix length cuts both the positions counted and the neighbours looked at
    assert orc.reconvergence_count(z, y, np.array([2, 2, 2, 2, 2])).tolist() == [2, 1, 1, 0, 0]
    assert orc.reconvergence_count(z, y, np.zeros(5, dtype=int)).tolist() == [0] * 5


def test_reconvergence_against_a_set_formulation_exhaustive():
    """All z, y over a 3-letter alphabet with L = 4: position q counts iff y_q is in the set
    {z_j : |j - q| <= 1, 0 <= j < L}."""
    L = 4
    for zt in itertools.product(range(3), repeat=L):
        zz = np.array([zt])
        for yt in itertools.product(range(3), repeat=L):
            want = sum(1 for q in range(L) if yt[q] in {zt[j] for j in range(max(0, q - 1), min(L, q + 2))})
            assert int(orc.reconvergence_count(zz, np.array([yt]), np.array([L]))[0]) == want


# ----------------------------------------------------------------------------- stochastic verification
def test_stochastic_accept_rule_by_hand_and_limits():
    W, page = 4, 16
    bt = np.arange(8).reshape(1, 8)
    L = np.array([5])
    tgt = np.array([[10, 11, 12, 13, 14]])
    run = lambda p, q, u, nf=0: orc.verify_accept_stochastic(np.array([p]), np.array([q]), np.array([u]), tgt, L, bt, page, nf)
    # p >= q: always accepted whatever u in [0, 1)
    r = run([0.5, 0.5, 0.5, 0.5], [0.5, 0.4, 0.1, 0.5], [0.999, 0.999, 0.999, 0.999])
    assert r["accept_len"][0] == 4 and r["bonus"][0] == 14
    # row 2: p/q = 0.25, u = 0.3 -> rejected; later rows do not count even though they would pass
    r = run([0.5, 0.5, 0.1, 0.9], [0.5, 0.5, 0.4, 0.1], [0.0, 0.9, 0.3, 0.0])
    assert r["accept_len"][0] == 2 and r["bonus"][0] == 12
    assert r["carry_slot"].tolist() == [-1, -1, 0, 1] and r["commit_slot"].tolist() == [5, 6, -1, -1]
    # same row with u = 0.2 < 0.25 -> accepted
    r = run([0.5, 0.5, 0.1, 0.9], [0.5, 0.5, 0.4, 0.1], [0.0, 0.9, 0.2, 0.0])
    assert r["accept_len"][0] == 4
    # p = 0 is never accepted (u * q < 0 is false), unless the row is the forced anchor
    assert run([0.0, 1, 1, 1], [0.3, 1, 1, 1], [0.0, 0, 0, 0])["accept_len"][0] == 0
    assert run([0.0, 1, 1, 1], [0.3, 1, 1, 1], [0.0, 0, 0, 0], nf=1)["accept_len"][0] == 4


def test_stochastic_acceptance_frequency_is_min_1_p_over_q():
    """Over many uniform draws a one-row window is accepted with frequency min(1, p/q)."""
    rng = np.random.default_rng(0)
    n = 40000
    bt = np.zeros((n, 2), dtype=np.int64)
    tgt = np.zeros((n, 2), dtype=np.int64)
    for p, q in ((0.2, 0.8), (0.6, 0.3), (0.05, 0.5)):
        u = rng.random((n, 1), dtype=np.float32)
        r = orc.verify_accept_stochastic(np.full((n, 1), p), np.full((n, 1), q), u, tgt, np.zeros(n, dtype=int), bt, 16, 0)
        freq = r["accept_len"].mean()
        assert abs(freq - min(1.0, p / q)) < 4 * math.sqrt(0.25 / n)


def test_stochastic_rule_with_degenerate_probabilities_is_the_greedy_rule():
    """p in {0, 1} with q = 1: the coin never matters and the rule is 'draft equals target'."""
    wl = synth.scaled(synth.workload("cfg1"), S=6, ctx=(10, 50))
    lay = synth.make_layout(wl, 3)
    rd = synth.make_round(wl, 3, 0)
    match = (rd["draft"] == rd["target"][:, :wl.shape.W]).astype(np.float32)
    u = np.random.default_rng(1).random(match.shape, dtype=np.float32)
    a = orc.verify_accept_stochastic(match, np.ones_like(match), u, rd["target"], lay["committed_len"], lay["block_table"], 16, 1)
    b = orc.verify_accept(rd["draft"], rd["target"], lay["committed_len"], lay["block_table"], 16, 1)
    for k in b:
        assert np.array_equal(a[k], b[k])


# ----------------------------------------------------------------------------- sampling head
def _mix32_py(x):
    x &= 0xFFFFFFFF
    x ^= x >> 16; x = (x * 0x85EBCA6B) & 0xFFFFFFFF
    x ^= x >> 13; x = (x * 0xC2B2AE35) & 0xFFFFFFFF
    x ^= x >> 16
    return x


def test_counter_uniform_against_plain_python_integers_and_statistics():
    seed, step = 0x1234567890ABCDEF, 7
    rows, cols = np.array([[0], [3], [511]]), np.array([[0, 1, 151935, 77777]])
    U = orc.counter_uniform(seed, step, rows, cols)
    for i, r in enumerate(rows[:, 0]):
        for j, c in enumerate(cols[0]):
            h = _mix32_py((seed & 0xFFFFFFFF) ^ 0x9E3779B9)
            h = _mix32_py(h + (seed >> 32))
            h = _mix32_py(h + step)
            h = _mix32_py(h + int(r))
            h = _mix32_py(h + int(c))
            assert U[i, j] == ((h >> 9) + 0.5) / 2 ** 23
    # the finaliser's published test value: mix(1) = 0x514E28B7
    assert _mix32_py(1) == 0x514E28B7
    # open interval, exactly representable in float32, flat histogram, no visible row/column correlation
    big = orc.counter_uniform(1, 0, np.arange(64)[:, None], np.arange(4096)[None, :])
    assert big.min() > 0 and big.max() < 1 and np.array_equal(big.astype(np.float32).astype(np.float64), big)
    hist = np.histogram(big, bins=16, range=(0, 1))[0] / big.size
    assert np.abs(hist - 1 / 16).max() < 0.004
    assert abs(np.corrcoef(big[:-1].ravel(), big[1:].ravel())[0, 1]) < 0.01
    assert abs(np.corrcoef(big[:, :-1].ravel(), big[:, 1:].ravel())[0, 1]) < 0.01
    assert not np.array_equal(big, orc.counter_uniform(1, 1, np.arange(64)[:, None], np.arange(4096)[None, :]))


def test_gumbel_max_sample_follows_the_softmax_and_reports_its_probability():
    """Draw the same 3 rows over 4000 steps: token frequencies match softmax(logits); q_tok is the
    softmax probability of the drawn token; lse is the log of the partition sum."""
    wl = synth.scaled(synth.workload("cfg1"), vocab=12)
    cfg = oracle_config(wl.shape)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 2))
    w["emb"] = w["emb"] * 5.0                        # a peaked but not degenerate distribution
    x = np.random.default_rng(0).standard_normal((3, cfg.d_model))
    _, _, logits = orc.lm_head_argmax(x, w, cfg)
    sm = torch.softmax(torch.from_numpy(logits), dim=1).numpy()
    counts = np.zeros_like(sm)
    n = 4000
    for step in range(n):
        tok, q, lse, _ = orc.lm_head_sample(x, w, cfg, seed=99, step=step)
        counts[np.arange(3), tok] += 1
        assert np.allclose(q, sm[np.arange(3), tok], rtol=1e-12)
        assert np.allclose(lse, torch.logsumexp(torch.from_numpy(logits), dim=1).numpy(), rtol=1e-12)
    assert 0.05 < sm.max() < 0.95
    assert np.abs(counts / n - sm).max() < 4 * math.sqrt(0.25 / n)


def test_rank_of_a_reference_token_sort_position_argmax_and_recall():
    """lm_head_rank against a stable sort (torch), the argmax (rank 0), hand-planted ties and the
    Recall@k reading of Section 5.1 (a hit iff rank < k: monotone in k, certain at k = V)."""
    wl = synth.scaled(synth.workload("cfg1"), vocab=40)
    cfg = oracle_config(wl.shape)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 5))
    rng = np.random.default_rng(3)
    R, V = 9, 40
    x = rng.standard_normal((R, cfg.d_model))
    ref = rng.integers(0, V, size=R)
    tok, _, logits = orc.lm_head_argmax(x, w, cfg)
    rank, ref_logit, lo, hi = orc.lm_head_rank(x, ref, w, cfg, tol=0.0)
    # position of the reference token in a descending stable sort (ties keep index order)
    order = torch.sort(torch.from_numpy(-logits), dim=1, stable=True).indices.numpy()
    for r in range(R):
        assert rank[r] == int(np.where(order[r] == ref[r])[0][0])
        assert ref_logit[r] == logits[r, ref[r]]
    assert np.array_equal(lo, rank) and np.array_equal(hi, rank)          # no exact ties in random data
    # the argmax has rank 0, and only it
    r0, _, _, _ = orc.lm_head_rank(x, tok, w, cfg)
    assert np.array_equal(r0, np.zeros(R, dtype=np.int32))
    assert ((rank == 0) == (ref == tok)).all()
    # planted ties: identical embedding rows give identical logits; the lower index ranks first
    w2 = dict(w); w2["emb"] = w["emb"].copy()
    w2["emb"][7] = w2["emb"][3]; w2["emb"][21] = w2["emb"][3]
    ra, _, _, _ = orc.lm_head_rank(x, np.full(R, 3), w2, cfg)
    rb, _, _, _ = orc.lm_head_rank(x, np.full(R, 7), w2, cfg)
    rc, _, lo_c, hi_c = orc.lm_head_rank(x, np.full(R, 21), w2, cfg, tol=1e-9)
    assert np.array_equal(rb, ra + 1) and np.array_equal(rc, ra + 2)
    assert np.array_equal(lo_c, ra) and np.array_equal(hi_c, ra + 2)      # the window spans the tie group
    # Recall@k = mean(rank < k): monotone in k, 1 at k = V; Recall@1 = agreement with the argmax
    rec = [float((rank < k).mean()) for k in range(1, V + 1)]
    assert all(b >= a for a, b in zip(rec, rec[1:])) and rec[-1] == 1.0
    assert rec[0] == float((ref == tok).mean())
    # brute force over rows and vocabulary, plain Python
    for r in range(R):
        cnt = 0
        for v in range(V):
            if v != ref[r] and (logits[r, v] > logits[r, ref[r]] or (logits[r, v] == logits[r, ref[r]] and v < ref[r])):
                cnt += 1
        assert cnt == rank[r]


# ----------------------------------------------------------------------------- other ways to mark rejected rows
def test_carry_variants_relate_as_they_must():
    """'none' is the embedding variant with E_carry = 0; 'projector' with F_rej = F is 'none';
    with another F_rej only the rejected rows change, and they are exactly F_rej h (one-hot probes)."""
    base = synth.scaled(synth.workload("cfg1"), S=2, ctx=(10, 40), hidden_norm=False)
    wl_n, wl_p = synth.scaled(base, carry_variant="none"), synth.scaled(base, carry_variant="projector")
    w = orc.prepare_weights(synth.make_weights(wl_p.shape, 3))
    rd = synth.make_round(base, 3, 0)
    lay = synth.make_layout(base, 3)
    split = orc.verify_accept(rd["draft"], rd["target"], lay["committed_len"], lay["block_table"], 16, 1)
    W = base.shape.W
    rejected = (np.tile(np.arange(W), base.S) >= np.repeat(split["accept_len"], W))
    assert rejected.any() and (~rejected).any()
    Z_e = orc.fuse_features(rd["H"], rejected, w, oracle_config(base.shape))
    w0 = dict(w); w0["e_carry"] = np.zeros_like(w["e_carry"])
    Z_e0 = orc.fuse_features(rd["H"], rejected, w0, oracle_config(base.shape))
    Z_n = orc.fuse_features(rd["H"], rejected, w, oracle_config(wl_n.shape))
    assert np.array_equal(Z_n, Z_e0) and not np.array_equal(Z_n, Z_e)
    wp = dict(w); wp["fc_rej"] = w["fc"]
    assert np.array_equal(orc.fuse_features(rd["H"], rejected, wp, oracle_config(wl_p.shape)), Z_n)
    Z_p = orc.fuse_features(rd["H"], rejected, w, oracle_config(wl_p.shape))
    assert np.array_equal(Z_p[~rejected], Z_n[~rejected]) and not np.allclose(Z_p[rejected], Z_n[rejected])
    r = int(np.flatnonzero(rejected)[0])
    want = [sum(w["fc_rej"][i, k] * float(rd["H"][r, k]) for k in range(base.shape.d_in)) for i in range(4)]
    assert np.allclose(Z_p[r, :4], want, atol=1e-12)


# ----------------------------------------------------------------------------- retention beyond one round
def test_carry_retention_holds_exactly_the_last_k_rounds_in_order():
    """After every round U must be the rejected rows of the last k rounds, oldest first, each row
    equal to the K/V the projection made for it in ITS round (positions kept)."""
    for k in (1, 2, 3):
        wl = synth.scaled(synth.workload("cfg1"), S=2, ctx=(10, 40), carry_rounds=k, n_rounds=8)
        cfg, st, _ = oracle_state(wl, 9)
        w = orc.prepare_weights(synth.make_weights(wl.shape, 9))
        segs = [[], []]                                   # per sequence: list of (K rows, V rows) per round
        for r in range(6):
            rd = synth.make_round(wl, 9, r)
            res = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY)
            for s in range(2):
                m = int(res["split"]["accept_len"][s])
                rows = slice(s * cfg.W + m, (s + 1) * cfg.W)
                segs[s].append(res["J"][:, rows])            # [Ld, W - m, 2, n_kv, hd]
                want = np.concatenate(segs[s][-k:], axis=1)
                c = int(st.carry_len[s])
                assert c == want.shape[1] == sum(st.carry_hist[s]) and len(st.carry_hist[s]) <= k
                got = np.transpose(st.carry[:, s, :, :, :c, :], (0, 3, 2, 1, 4))       # -> [Ld, c, 2, n_kv, hd]
                assert np.array_equal(got, want)
                assert np.isnan(st.carry[:, s, :, :, c:, :]).all()
        assert max(int(x) for x in st.carry_len) <= k * cfg.W


def test_retained_rows_change_the_next_draft_and_k1_is_the_papers_round():
    wl1 = synth.scaled(synth.workload("cfg1"), S=2, ctx=(10, 40), n_rounds=6)
    wl2 = synth.scaled(wl1, carry_rounds=2)
    w = orc.prepare_weights(synth.make_weights(wl1.shape, 4))
    w["wo"] = w["wo"] * 40.0
    _, st1, _ = oracle_state(wl1, 4)
    _, st2, _ = oracle_state(wl2, 4)
    differs = False
    for r in range(4):
        rd = synth.make_round(wl1, 4, r)
        a = orc.draft_round(rd["draft"], rd["target"], rd["H"], st1, w, 1, orc.MODE_CARRY)
        b = orc.draft_round(rd["draft"], rd["target"], rd["H"], st2, w, 1, orc.MODE_CARRY)
        assert np.array_equal(st1.pool, st2.pool)                      # the committed cache never depends on U
        if r == 0:
            assert np.array_equal(a["x_final"], b["x_final"])          # nothing older to retain yet
        else:
            differs |= np.abs(a["x_final"] - b["x_final"]).max() > 1e-6
    assert differs



# ----------------------------------------------------------------------------- the storage-rounded diagnostic mode
def test_storage_rounded_mode_changes_nothing_unless_asked_and_rounds_where_it_says():
    """round_store = identity is the exact oracle bit for bit; a bfloat16 round_store is called on the
    tensors an implementation with bf16 hand-offs stores (z, cached K and V per layer, a, rotated q / k_b,
    v_b, o per layer, b and the gated activation per layer, y), and moves the result by bf16-sized amounts only."""
    wl = _full_layer_workload(qk_norm=False)
    w = orc.prepare_weights(synth.make_weights(wl.shape, 3))
    rd = synth.make_round(wl, 3, 0)
    runs = {}
    calls = []

    def bf16(x):
        calls.append(np.shape(x))
        return synth.round_bf16(np.asarray(x, dtype=np.float32)).astype(np.float64)

    for name, hook in (("exact", None), ("identity", lambda x: x), ("bf16", bf16)):
        _, st, _ = oracle_state(wl, 3)
        runs[name] = orc.draft_round(rd["draft"], rd["target"], rd["H"], st, w, 1, orc.MODE_CARRY, round_store=hook)
        runs[name]["pool"] = st.pool
    for k in ("x_final", "attn_out", "J", "tok"):
        assert np.array_equal(runs["exact"][k], runs["identity"][k], equal_nan=True)
    Ld, S = wl.shape.n_layers, wl.S
    # z, (K, V) per layer | per layer: a, then per sequence (q, k_b, v_b), o, b, act | y
    assert len(calls) == 1 + 2 * Ld + Ld * (1 + 3 * S + 1 + 2) + 1
    J = runs["bf16"]["J"]
    kept = ~np.isnan(J)
    assert np.array_equal(J[kept], synth.round_bf16(J[kept].astype(np.float32)).astype(np.float64))
    for k in ("x_final", "attn_out"):
        d = np.abs(runs["bf16"][k] - runs["exact"][k]).max() / np.abs(runs["exact"][k]).max()
        assert 1e-5 < d < 2e-2, (k, d)
