"""Seeded synthetic inputs for the Carryover drafting round.

This module only draws random numbers and shapes them: it holds none of the
method's arithmetic (no acceptance rule, projection, rotation, attention or
argmax).  Both the CPU oracle's tests and the CUDA path's tests feed on the
arrays made here, so the two sides see bit-identical inputs.

Every array is float32 / int32 numpy.  For ``dtype == "bf16"`` workloads the
floating-point arrays are rounded ONCE, here, to values that bfloat16 holds
exactly, so a later cast to bfloat16 (device side) or float64 (oracle side)
loses nothing.

Each tensor has its own generator stream ``default_rng([seed, stream, ...])``,
so any one of them (one pool layer, one round) can be drawn without the others.

The workloads stand in for the paper's evaluation (Section 4 and Appendix B:
5 captured target layers, 5 drafter layers, 15 proposals + anchor, concurrency
1..32, generation caps of 1-2k tokens after a prompt); the prompts, trained
drafters and target models themselves are not used.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np

_STREAM_WEIGHTS = 1
_STREAM_LAYOUT = 2
_STREAM_POOL = 3
_STREAM_ROUND = 4


@dataclass(frozen=True)
class DrafterShape:
    """Static sizes of the drafter and of the target features it consumes."""

    dtype: str            # "f32" or "bf16": storage type of weights, H and KV
    d_target: int         # width of one captured target layer
    n_cap: int            # captured target layers (D_in = d_target * n_cap)
    d_model: int          # drafter width D (= n_q * hd)
    n_layers: int         # drafter layers Ld
    n_q: int
    n_kv: int
    hd: int
    vocab: int
    W: int                # rows of the verified window = block size
    page: int = 16
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6
    hidden_norm: bool = True
    h_rms: Optional[Tuple[float, float]] = None  # per-layer RMS range of H
    d_ff: int = 0         # width of the gated MLP of a drafter layer; 0 = attention sub-layer only
    qk_norm: bool = False # per-head RMS norm (with gain) of queries and keys before the rotation
    carry_variant: str = "embedding"  # how rejected rows are told apart: "embedding" (E_carry), "none", "projector"
    carry_rounds: int = 1 # rounds for which rejected rows stay in the carry slot (the paper's setting: 1)

    @property
    def d_in(self) -> int:
        return self.d_target * self.n_cap

    @property
    def mask_token_id(self) -> int:
        return self.vocab - 1


@dataclass(frozen=True)
class Workload:
    name: str
    shape: DrafterShape
    S: int                       # sequences in the batch
    ctx: Tuple[int, int]         # committed context L_s ~ integer-uniform [lo, hi]
    accept: Tuple                # ("rej_uniform", lo, hi) | ("geom", mean) | ("fixed_m", m)
    n_forced: int                # 1: row 0 is the anchor and always accepted
    n_rounds: int
    spare_pages: int = 8         # pages per sequence beyond what n_rounds can fill

    @property
    def R(self) -> int:
        return self.S * self.shape.W

    def max_pages_per_seq(self) -> int:
        sh = self.shape
        grow = (self.n_rounds + 1) * sh.W
        return (self.ctx[1] + grow + sh.page - 1) // sh.page + self.spare_pages


_TINY = DrafterShape(dtype="f32", d_target=256, n_cap=2, d_model=256, n_layers=1,
                     n_q=4, n_kv=2, hd=64, vocab=1024, W=8, rope_theta=1.0e4)
_FULL = DrafterShape(dtype="bf16", d_target=4096, n_cap=5, d_model=4096, n_layers=5,
                     n_q=32, n_kv=8, hd=128, vocab=151936, W=16, rope_theta=1.0e6,
                     h_rms=(0.5, 4.0))


def workload(name: str) -> Workload:
    """The five named configurations (tiny fp32; batch 1; batch 32; long context; sweep base)."""
    if name == "cfg1":
        return Workload("cfg1", _TINY, S=1, ctx=(128, 128), accept=("rej_uniform", 0, 7),
                        n_forced=1, n_rounds=16)
    if name == "cfg2":
        return Workload("cfg2", _FULL, S=1, ctx=(2048, 2048), accept=("geom", 6.0),
                        n_forced=1, n_rounds=64)
    if name == "cfg3":
        return Workload("cfg3", _FULL, S=32, ctx=(512, 8192), accept=("geom", 6.0),
                        n_forced=1, n_rounds=64)
    if name == "cfg4":
        return Workload("cfg4", replace(_FULL, W=32), S=4, ctx=(32768, 32768),
                        accept=("geom", 10.0), n_forced=1, n_rounds=16)
    if name == "cfg5":
        return Workload("cfg5", _FULL, S=1, ctx=(4096, 4096), accept=("fixed_m", 8),
                        n_forced=0, n_rounds=16)
    if name in ("cfg2f", "cfg3f"):
        # the same batches with a complete drafter layer: gated MLP of width 9728 and q/k norms
        base = workload(name[:-1])
        return replace(base, name=name, shape=replace(base.shape, d_ff=9728, qk_norm=True))
    if name == "cfg3p":
        # batch 32 with the separate projector for rejected rows (Section 5, Table 4(b)) instead of the embedding
        base = workload("cfg3")
        return replace(base, name=name, shape=replace(base.shape, carry_variant="projector"))
    raise KeyError(name)


def sweep_point(S: int, W: int, m: int, n_forced: int = 0, n_rounds: int = 16) -> Workload:
    """One point of the overhead sweep: context 4096, fixed accepted rows m."""
    return Workload(f"cfg5_S{S}_W{W}_m{m}", replace(_FULL, W=W), S=S, ctx=(4096, 4096),
                    accept=("fixed_m", m), n_forced=n_forced, n_rounds=n_rounds)


def scaled(wl: Workload, **kw) -> Workload:
    """A copy of a workload with some shape / batch fields replaced (test sizes)."""
    shape_keys = {k: v for k, v in kw.items() if hasattr(wl.shape, k) and k != "name"}
    wl_keys = {k: v for k, v in kw.items() if k not in shape_keys}
    return replace(wl, shape=replace(wl.shape, **shape_keys), **wl_keys)


# --------------------------------------------------------------------------- storage rounding
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_bf16(x) if dtype == "bf16" else x


def _normal(rng: np.random.Generator, shape, scale: float = 1.0) -> np.ndarray:
    out = rng.standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        out *= np.float32(scale)
    return out


# --------------------------------------------------------------------------- weights
_WEIGHT_ORDER = ("fc", "e_carry", "g_hidden", "wk", "wv", "wq", "wo", "g_attn", "g_final", "emb",
                 "w_gate", "w_up", "w_down", "g_mlp", "g_qnorm", "g_knorm", "fc_rej")   # new names go last: stream index = position


def weight_shapes(sh: DrafterShape) -> Dict[str, Tuple[int, ...]]:
    D, Ld = sh.d_model, sh.n_layers
    out = {
        "fc": (D, sh.d_in),
        "e_carry": (sh.d_in,),
        "g_hidden": (D,),
        "wk": (Ld, sh.n_kv * sh.hd, D),
        "wv": (Ld, sh.n_kv * sh.hd, D),
        "wq": (Ld, sh.n_q * sh.hd, D),
        "wo": (Ld, D, sh.n_q * sh.hd),
        "g_attn": (Ld, D),
        "g_final": (D,),
        "emb": (sh.vocab, D),
    }
    if sh.d_ff > 0:
        out.update({"w_gate": (Ld, sh.d_ff, D), "w_up": (Ld, sh.d_ff, D), "w_down": (Ld, D, sh.d_ff),
                    "g_mlp": (Ld, D)})
    if sh.qk_norm:
        out.update({"g_qnorm": (Ld, sh.hd), "g_knorm": (Ld, sh.hd)})
    if sh.carry_variant == "projector":
        out["fc_rej"] = (D, sh.d_in)
    return out


def make_weights(sh: DrafterShape, seed: int) -> Dict[str, np.ndarray]:
    """Matrices and the embedding ~ N(0, 0.02); norm gains 1 + 0.1 N(0,1); E_carry ~ N(0,1)."""
    out = {}
    shapes = weight_shapes(sh)
    for i, name in enumerate(_WEIGHT_ORDER):
        if name not in shapes:
            continue
        rng = np.random.default_rng([seed, _STREAM_WEIGHTS, i])
        if name.startswith("g_"):
            w = np.float32(1.0) + _normal(rng, shapes[name], 0.1)
        elif name == "e_carry":
            w = _normal(rng, shapes[name], 1.0)
        else:
            w = _normal(rng, shapes[name], 0.02)
        out[name] = to_storage(w, sh.dtype)
    return out


# --------------------------------------------------------------------------- paged state layout
def make_layout(wl: Workload, seed: int) -> Dict[str, np.ndarray]:
    """Committed lengths and a page table whose physical pages are a random permutation."""
    sh = wl.shape
    rng = np.random.default_rng([seed, _STREAM_LAYOUT])
    lo, hi = wl.ctx
    committed_len = rng.integers(lo, hi + 1, size=wl.S).astype(np.int32)
    mp = wl.max_pages_per_seq()
    n_pages = wl.S * mp
    perm = rng.permutation(n_pages).astype(np.int32)
    block_table = perm.reshape(wl.S, mp)
    return {"committed_len": committed_len, "block_table": block_table,
            "n_pages": np.int32(n_pages), "max_pages_per_seq": np.int32(mp)}


def pool_layer(wl: Workload, seed: int, layer: int, n_pages: int) -> np.ndarray:
    """N(0,1) contents of one layer of the KV pool, [n_pages, n_kv, 2, page, hd]."""
    sh = wl.shape
    rng = np.random.default_rng([seed, _STREAM_POOL, layer])
    return to_storage(_normal(rng, (n_pages, sh.n_kv, 2, sh.page, sh.hd)), sh.dtype)


# --------------------------------------------------------------------------- per-round inputs
def draw_accept(wl: Workload, rng: np.random.Generator) -> np.ndarray:
    """Accepted window rows m_s per sequence, following the workload's acceptance recipe."""
    W = wl.shape.W
    kind = wl.accept[0]
    if kind == "rej_uniform":
        rej = rng.integers(wl.accept[1], wl.accept[2] + 1, size=wl.S)
        m = W - rej
    elif kind == "geom":
        p = 1.0 / (1.0 + float(wl.accept[1]))
        g = rng.geometric(p, size=wl.S) - 1          # support 0, 1, 2, ...
        m = np.minimum(g, W - 1) + 1                  # anchor row + accepted proposals
    elif kind == "fixed_m":
        m = np.full(wl.S, int(wl.accept[1]))
    else:
        raise ValueError(kind)
    return m.astype(np.int32)


def make_tokens(wl: Workload, rng: np.random.Generator, m: np.ndarray):
    """draft [S,W] and aligned target [S,W+1] tokens that realise the accepted lengths m."""
    sh = wl.shape
    V, W = sh.vocab, sh.W
    draft = rng.integers(0, V, size=(wl.S, W)).astype(np.int64)
    target = rng.integers(0, V, size=(wl.S, W + 1)).astype(np.int64)
    bump = rng.integers(1, V, size=wl.S).astype(np.int64)
    for s in range(wl.S):
        ms = int(m[s])
        target[s, :ms] = draft[s, :ms]
        if ms < W:
            target[s, ms] = (draft[s, ms] + bump[s]) % V      # differs for certain
    return draft.astype(np.int32), target.astype(np.int32)


def make_hidden(wl: Workload, rng: np.random.Generator) -> np.ndarray:
    """Concatenated target hiddens H [S*W, D_in]; captured layer i has its own RMS."""
    sh = wl.shape
    H = _normal(rng, (wl.R, sh.n_cap, sh.d_target))
    if sh.h_rms is not None:
        lo, hi = sh.h_rms
        for i in range(sh.n_cap):
            r = lo + (hi - lo) * (i / max(sh.n_cap - 1, 1))
            H[:, i, :] *= np.float32(r)
    return to_storage(H.reshape(wl.R, sh.d_in), sh.dtype)


def make_round(wl: Workload, seed: int, r: int) -> Dict[str, np.ndarray]:
    """Inputs of round r: draft, target, H, and the accepted lengths they realise."""
    rng = np.random.default_rng([seed, _STREAM_ROUND, r])
    m = draw_accept(wl, rng)
    draft, target = make_tokens(wl, rng, m)
    H = make_hidden(wl, rng)
    return {"draft": draft, "target": target, "H": H, "m": m}
