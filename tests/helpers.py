"""Glue shared by the tests: turns synthetic workloads into oracle objects."""
from __future__ import annotations

import numpy as np

from oracle import cod_oracle as orc
from paper_2609_14717_b200 import synth


def oracle_config(sh: synth.DrafterShape) -> orc.OracleConfig:
    return orc.OracleConfig(
        d_target=sh.d_target, n_cap=sh.n_cap, d_model=sh.d_model, n_layers=sh.n_layers,
        n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, vocab=sh.vocab, mask_token_id=sh.mask_token_id,
        W=sh.W, page=sh.page, rope_theta=sh.rope_theta, rms_eps=sh.rms_eps,
        hidden_norm=sh.hidden_norm, d_ff=sh.d_ff, qk_norm=sh.qk_norm, carry_variant=sh.carry_variant, carry_rounds=sh.carry_rounds)


def oracle_state(wl: synth.Workload, seed: int, fill_pool: bool = True):
    """Oracle state with the synthetic layout and (optionally) a pre-filled pool."""
    cfg = oracle_config(wl.shape)
    lay = synth.make_layout(wl, seed)
    st = orc.OracleState(cfg, wl.S, int(lay["n_pages"]), lay["block_table"], lay["committed_len"])
    if fill_pool:
        for l in range(cfg.n_layers):
            st.pool[l] = synth.pool_layer(wl, seed, l, int(lay["n_pages"]))
    return cfg, st, lay


def small_bf16(S=2, W=16, n_layers=2, ctx=(40, 90), **kw) -> synth.Workload:
    """A scaled-down bf16 workload with the full config's head geometry (hd 128, GQA 4:1)."""
    base = synth.workload("cfg3")
    args = dict(S=S, W=W, n_layers=n_layers, ctx=ctx, d_target=256, n_cap=2, d_model=512,
                n_q=4, n_kv=1, vocab=1000, n_rounds=4)
    args.update(kw)
    return synth.scaled(base, **args)


def rel_err(a: np.ndarray, ref: np.ndarray) -> float:
    """max |a - ref| / max |ref| over one tensor."""
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.max(np.abs(ref))
    return float(np.max(np.abs(a - ref)) / (den if den > 0 else 1.0))
