"""cod_lm_head_argmax_static — the LM-head argmax for callers that are not allowed to allocate
device memory (a server whose pool owns all of it, a loop that cannot take cudaMalloc's
device-wide synchronisation). Its scratch is a fixed array inside the library, shared by every
call on the device and never cleared between calls, so this test calls it twice in a row with
different inputs and checks each result against the ordinary entry point (cod_lm_head_argmax),
which uses the context's own workspace. Collected last on purpose: a run that stops at the first
failure has then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import cod_oracle as orc
from paper_2609_14717_b200 import synth
from tests.helpers import oracle_config, small_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_argmax_matches_the_context_path_twice_in_a_row(dtype):
    from paper_2609_14717_b200 import binding as B
    wl = small_bf16(S=1, vocab=3000, d_model=512) if dtype == "bf16" else synth.workload("cfg1")
    sh = wl.shape
    w = synth.make_weights(sh, 21)
    cfg = B.make_config(sh, 8, 4, 8)
    ctx = B.Context(cfg)
    w_dev = B.weights_to_device(w, sh.dtype)
    ctx.set_weights(w_dev)
    gen = torch.Generator(device="cuda").manual_seed(5)
    w_o = {"g_final": np.asarray(w["g_final"], dtype=np.float64), "emb": np.asarray(w["emb"], dtype=np.float64)}
    tol = 2e-2 if dtype == "bf16" else 1e-3
    for n_rows in (48, 7):                                     # two calls in a row, the second smaller
        x = torch.randn(n_rows, sh.d_model, generator=gen, device="cuda")
        tok_ref = torch.zeros(n_rows, dtype=torch.int32, device="cuda")
        top_ref = torch.zeros(n_rows, dtype=torch.float32, device="cuda")
        ctx_rows = min(n_rows, 8 * sh.W)
        ctx.lm_head_argmax(x[:ctx_rows].contiguous(), ctx_rows, tok_ref, top_ref)
        tok = torch.full((n_rows,), -1, dtype=torch.int32, device="cuda")
        top = torch.zeros(n_rows, dtype=torch.float32, device="cuda")
        B.lm_head_argmax_static(w_dev["emb"], w_dev["g_final"], x, tok, top, sh.rms_eps)
        torch.cuda.synchronize()
        # same kernels on the same inputs: identical tokens and logits (tolerance of the parity tests)
        assert torch.equal(tok[:ctx_rows], tok_ref[:ctx_rows])
        ref = top_ref[:ctx_rows].cpu().numpy()
        assert np.max(np.abs(top[:ctx_rows].cpu().numpy() - ref)) <= (2e-2 if dtype == "bf16" else 1e-3) * np.max(np.abs(ref))
        assert (tok >= 0).all() and (tok < sh.vocab).all()
        # and against the CPU oracle's LM head on all rows: tokens where its top-2 gap is clear, top logit to tolerance
        t_o, gap, logits = orc.lm_head_argmax(x.cpu().numpy().astype(np.float64), w_o, oracle_config(sh))
        sure = gap >= 1e-2
        assert sure.sum() >= n_rows // 2
        assert np.array_equal(tok.cpu().numpy()[sure], t_o[sure])
        assert np.max(np.abs(top.cpu().numpy() - logits.max(axis=1))) <= tol * np.max(np.abs(logits))
    # beyond the fixed capacity: refused, nothing launched
    big = torch.zeros(65, sh.d_model, device="cuda")
    with pytest.raises(B.CodError) as e:
        B.lm_head_argmax_static(w_dev["emb"], w_dev["g_final"], big, torch.zeros(65, dtype=torch.int32, device="cuda"),
                                None, sh.rms_eps)
    assert e.value.status == -6
    ctx.close()


def test_static_scratch_argmax_at_its_size_limits_against_the_oracle():
    """Exactly 64 rows x 8192 columns (the whole scratch in use, the wide-row kernels), twice in a row; one
    column group beyond the limit is refused."""
    from paper_2609_14717_b200 import binding as B
    D, V, R = 8192, 1536, 64
    rng = np.random.default_rng(31)
    emb = synth.round_bf16(rng.standard_normal((V, D), dtype=np.float32) * np.float32(0.02))
    g = synth.round_bf16(np.float32(1.0) + np.float32(0.1) * rng.standard_normal(D, dtype=np.float32))
    emb_d, g_d = B.to_device(emb, "bf16"), B.to_device(g, "bf16")
    sh = synth.scaled(synth.workload("cfg3"), d_model=D, vocab=V).shape
    w_o = {"g_final": g.astype(np.float64), "emb": emb.astype(np.float64)}
    for rep in range(2):
        x = rng.standard_normal((R, D), dtype=np.float32)
        tok = torch.full((R,), -1, dtype=torch.int32, device="cuda")
        top = torch.zeros(R, dtype=torch.float32, device="cuda")
        B.lm_head_argmax_static(emb_d, g_d, torch.from_numpy(x).cuda(), tok, top, sh.rms_eps)
        torch.cuda.synchronize()
        t_o, gap, logits = orc.lm_head_argmax(x.astype(np.float64), w_o, oracle_config(sh))
        sure = gap >= 1e-2
        assert sure.sum() >= R // 2
        assert np.array_equal(tok.cpu().numpy()[sure], t_o[sure])
        assert np.max(np.abs(top.cpu().numpy() - logits.max(axis=1))) <= 2e-2 * np.max(np.abs(logits))
    wide = torch.zeros(R, D + 8, device="cuda")
    with pytest.raises(B.CodError) as e:
        B.lm_head_argmax_static(torch.zeros(V, D + 8, dtype=torch.bfloat16, device="cuda"),
                                torch.ones(D + 8, dtype=torch.bfloat16, device="cuda"), wide,
                                torch.zeros(R, dtype=torch.int32, device="cuda"), None, sh.rms_eps)
    assert e.value.status == -6
