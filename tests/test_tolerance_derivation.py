"""Where the whole-round tolerance of the full-size GPU test comes from, measured on the CPU.

An implementation that hands bfloat16 tensors from step to step (fused features, normalised activations,
q / k / v, attention outputs) cannot agree with the exact float64 oracle to the single-step bound in the
deeper drafter layers, and not with ANOTHER such implementation either: the oracle's storage-rounded mode,
run twice with pre-rounding values that differ by 3e-7 relative (what float32 accumulation in a different
order does), gives two results as far from each other as each is from the exact one.  The full-size
drafter shapes are used (five layers, width 4096, context 2048); only the vocabulary is cut down, the LM
head plays no part here."""
import copy

import numpy as np

from oracle import cod_oracle as orc
from paper_2609_14717_b200 import synth
from tests.helpers import oracle_config, oracle_state, rel_err


def test_bf16_hand_offs_move_the_deeper_layers_by_percent_and_do_not_cancel():
    wl = synth.scaled(synth.workload("cfg2"), vocab=4096, n_rounds=4)
    sh = wl.shape
    cfg, st, _ = oracle_state(wl, 11)
    w = orc.prepare_weights(synth.make_weights(sh, 11))
    jitter = np.random.default_rng(0)

    def bf16(x):
        return synth.round_bf16(np.asarray(x, dtype=np.float32)).astype(np.float64)

    def bf16_after_jitter(x):
        x = np.asarray(x, dtype=np.float64)
        return bf16(x * (1.0 + 3e-7 * jitter.standard_normal(x.shape)))

    hooks = {"exact": None, "a": bf16, "b": bf16_after_jitter}
    states = {k: copy.deepcopy(st) for k in hooks}
    worst = {"a-exact": 0.0, "b-exact": 0.0, "a-b": 0.0, "layer0": 0.0}
    for r in range(2):
        rd = synth.make_round(wl, 11, r)
        res = {k: orc.draft_round(rd["draft"], rd["target"], rd["H"], states[k], w, wl.n_forced, orc.MODE_CARRY,
                                  round_store=h) for k, h in hooks.items()}
        worst["layer0"] = max(worst["layer0"], rel_err(res["a"]["attn_out"][0], res["exact"]["attn_out"][0]))
        for l in range(1, sh.n_layers):
            worst["a-exact"] = max(worst["a-exact"], rel_err(res["a"]["attn_out"][l], res["exact"]["attn_out"][l]))
            worst["b-exact"] = max(worst["b-exact"], rel_err(res["b"]["attn_out"][l], res["exact"]["attn_out"][l]))
            worst["a-b"] = max(worst["a-b"], rel_err(res["a"]["attn_out"][l], res["b"]["attn_out"][l]))
    print(worst)
    assert worst["layer0"] < 2e-2                       # one layer deep the single-step bound holds
    assert 1e-2 < worst["a-exact"] < 5e-2 and 1e-2 < worst["b-exact"] < 5e-2
    assert worst["a-b"] > 0.3 * worst["a-exact"]        # the two realisations do not track each other
