"""ctypes binding of libcod.so (the C ABI declared in include/cod.h).

Argument marshalling only: every step of the round runs in the library's CUDA kernels.
torch is used for device memory and the current stream.  If the compiled library is
missing the import of this module fails — there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcod.so")

COD_F32, COD_BF16 = 0, 1
COD_CARRY, COD_BASELINE = 0, 1
COD_F_HIDDEN_NORM = 1
COD_F_NO_TENSOR_CORES = 2
COD_F_ATTN_ONE_ITEM_CTAS = 32
COD_F_ATTN_PERSISTENT = 64
COD_F_QK_NORM = 4
COD_F_NO_CARRY_EMBED = 8
COD_F_REJ_PROJECTOR = 16
DEV_BAD_TOKEN, DEV_PAGE_OVERFLOW, DEV_BAD_PAGE, DEV_TIMEOUT, DEV_BAD_LEN = 1, 2, 4, 8, 16

EXPORTS = ("cod_create", "cod_destroy", "cod_set_weights", "cod_verify_accept", "cod_project_kv",
           "cod_scatter_kv", "cod_block_attn", "cod_lm_head_argmax", "cod_lm_head_argmax_static",
           "cod_draft_round", "cod_reconvergence_count", "cod_verify_accept_stochastic",
           "cod_draft_round_stochastic", "cod_lm_head_sample", "cod_lm_head_rank",
           "cod_poll_status", "cod_set_wait_limit", "cod_selftest_expire_wait",
           "cod_profile_enable", "cod_profile_read", "cod_launch_count",
           "cod_workspace_bytes", "cod_error_string")
KERNEL_CLASSES = ("verify", "fc", "kv", "qkv", "attn", "oproj", "lmhead", "rowops", "mlp")


class CodConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "d_target", "n_cap", "d_model", "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "vocab",
        "mask_token_id", "block", "page_size", "max_batch", "max_pages_per_seq", "n_pages", "dtype")] + [
        ("flags", C.c_uint32), ("rope_theta", C.c_float), ("rms_eps", C.c_float),
        ("attn_split_len", C.c_int32), ("d_ff", C.c_int32), ("carry_rounds", C.c_int32)]


_WEIGHT_FIELDS = ("fc", "e_carry", "g_hidden", "wk", "wv", "wq", "wo", "g_attn", "g_final", "emb",
                  "w_gate", "w_up", "w_down", "g_mlp", "g_qnorm", "g_knorm",   # these six: complete layer only
                  "fc_rej")                                                     # separate-projector variant only
_SPLIT_FIELDS = ("accept_len", "bonus", "row_pos", "commit_slot", "carry_slot", "acc_rows", "acc_off",
                 "rej_rows", "rej_off")
_STATE_FIELDS = ("kv_pool", "block_table", "committed_len", "carry_kv", "carry_len", "carry_hist")
_TAP_FIELDS = ("z", "attn_out", "x_final", "top_logit", "carry_mass")


class CodWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WEIGHT_FIELDS]


class CodState(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _STATE_FIELDS]


class CodSplit(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _SPLIT_FIELDS]


class CodTaps(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _TAP_FIELDS]


def load_library() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int, C.c_int64
    lib.cod_create.argtypes = [C.POINTER(CodConfig), C.POINTER(vp)]
    lib.cod_destroy.argtypes = [vp]
    lib.cod_set_weights.argtypes = [vp, C.POINTER(CodWeights), vp]
    lib.cod_verify_accept.argtypes = [vp, vp, vp, i32, i32, C.POINTER(CodState), C.POINTER(CodSplit), vp]
    lib.cod_project_kv.argtypes = [vp, vp, C.POINTER(CodSplit), i32, i32, vp, vp]
    lib.cod_scatter_kv.argtypes = [vp, vp, C.POINTER(CodSplit), i32, i32, C.POINTER(CodState), vp]
    lib.cod_block_attn.argtypes = [vp, i32, vp, vp, vp, C.POINTER(CodState), i32, i32, vp, vp, vp]
    lib.cod_lm_head_argmax.argtypes = [vp, vp, i32, vp, vp, vp]
    lib.cod_lm_head_argmax_static.argtypes = [vp, vp, vp, i32, i32, i32, i32, C.c_float, vp, vp, vp]
    lib.cod_draft_round.argtypes = [vp, vp, vp, vp, i32, i32, i32, C.POINTER(CodState), C.POINTER(CodSplit),
                                    vp, C.POINTER(CodTaps), vp]
    lib.cod_reconvergence_count.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    lib.cod_lm_head_sample.argtypes = [vp, vp, i32, C.c_uint64, C.c_uint32, vp, vp, vp, vp]
    lib.cod_lm_head_rank.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.cod_verify_accept_stochastic.argtypes = [vp, vp, vp, vp, vp, i32, i32, C.POINTER(CodState), C.POINTER(CodSplit), vp]
    lib.cod_draft_round_stochastic.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, C.POINTER(CodState),
                                               C.POINTER(CodSplit), vp, C.POINTER(CodTaps), vp, C.c_uint64,
                                               C.c_uint32, vp]
    lib.cod_poll_status.argtypes = [vp, C.POINTER(C.c_uint32), i32, vp]
    lib.cod_profile_enable.argtypes = [vp, C.c_uint32]
    lib.cod_profile_read.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.cod_launch_count.argtypes = [vp]
    lib.cod_launch_count.restype = i64
    lib.cod_workspace_bytes.argtypes = [vp]
    lib.cod_workspace_bytes.restype = i64
    lib.cod_error_string.argtypes = [i32]
    lib.cod_error_string.restype = C.c_char_p
    for name in EXPORTS[:-3]:
        getattr(lib, name).restype = i32
    return lib


_LIB: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _LIB
    if _LIB is None:
        _LIB = load_library()
    return _LIB


class CodError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {lib().cod_error_string(status).decode()} ({status})")


def _check(fn: str, status: int) -> None:
    if status != 0:
        raise CodError(fn, status)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def torch_dtype(dtype: str):
    return torch.bfloat16 if dtype == "bf16" else torch.float32


def to_device(a: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    """Host float32 array (already holding storage-exact values) -> device tensor of the storage type."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(device=device, dtype=torch_dtype(dtype))


class Split:
    """Device arrays cod_verify_accept fills."""

    def __init__(self, S: int, W: int, device="cuda"):
        i32 = dict(dtype=torch.int32, device=device)
        self.accept_len = torch.zeros(S, **i32)
        self.bonus = torch.zeros(S, **i32)
        self.row_pos = torch.zeros(S * W, **i32)
        self.commit_slot = torch.zeros(S * W, **i32)
        self.carry_slot = torch.zeros(S * W, **i32)
        self.acc_rows = torch.zeros(S * W, **i32)
        self.acc_off = torch.zeros(S + 1, **i32)
        self.rej_rows = torch.zeros(S * W, **i32)
        self.rej_off = torch.zeros(S + 1, **i32)

    def struct(self) -> CodSplit:
        return CodSplit(*[_ptr(getattr(self, n)) for n in _SPLIT_FIELDS])

    def to_host(self) -> Dict[str, np.ndarray]:
        return {n: getattr(self, n).cpu().numpy() for n in _SPLIT_FIELDS}


class State:
    """Paged committed KV, block table, carry slot and lengths of one batch (device tensors)."""

    def __init__(self, cfg: CodConfig, dtype: str, S: int, block_table: np.ndarray, committed_len: np.ndarray,
                 device="cuda"):
        td = torch_dtype(dtype)
        self.S = S
        self.kv_pool = torch.zeros((cfg.n_layers, cfg.n_pages, cfg.n_kv_heads, 2, cfg.page_size, cfg.head_dim),
                                   dtype=td, device=device)
        self.block_table = torch.from_numpy(np.ascontiguousarray(block_table, dtype=np.int32)).to(device)
        self.committed_len = torch.from_numpy(np.ascontiguousarray(committed_len, dtype=np.int32)).to(device)
        k = max(1, int(cfg.carry_rounds))                       # rounds of rejected rows the carry slot holds
        self.carry_kv = torch.zeros((cfg.n_layers, cfg.max_batch, cfg.n_kv_heads, 2, k * cfg.block, cfg.head_dim),
                                    dtype=td, device=device)
        self.carry_len = torch.zeros(S, dtype=torch.int32, device=device)
        self.carry_hist = torch.zeros((S, k), dtype=torch.int32, device=device) if k > 1 else None

    def struct(self) -> CodState:
        return CodState(*[_ptr(getattr(self, n)) for n in _STATE_FIELDS])


class Taps:
    def __init__(self, cfg: CodConfig, S: int, device="cuda"):
        R = S * cfg.block
        f32 = dict(dtype=torch.float32, device=device)
        self.z = torch.zeros((R, cfg.d_model), **f32)
        self.attn_out = torch.zeros((cfg.n_layers, R, cfg.n_q_heads * cfg.head_dim), **f32)
        self.x_final = torch.zeros((R, cfg.d_model), **f32)
        self.top_logit = torch.zeros(R, **f32)
        self.carry_mass = torch.zeros((cfg.n_layers, S, cfg.block, cfg.n_q_heads), **f32)

    def struct(self) -> CodTaps:
        return CodTaps(*[_ptr(getattr(self, n)) for n in _TAP_FIELDS])


class Context:
    """Owns a cod_ctx on the current CUDA device; methods mirror the C entry points."""

    def __init__(self, cfg: CodConfig):
        if not torch.cuda.is_available():
            raise RuntimeError("the Carryover drafting library needs a CUDA device (no CPU fallback)")
        torch.cuda.init()
        torch.zeros(1, device="cuda")          # make sure the primary context exists
        self.cfg = cfg
        self.dtype = "bf16" if cfg.dtype == COD_BF16 else "f32"
        self._h = C.c_void_p()
        _check("cod_create", lib().cod_create(C.byref(cfg), C.byref(self._h)))
        self._weights = None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().cod_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- set-up
    def set_weights(self, w: Dict[str, torch.Tensor]) -> None:
        self._weights = {k: w[k] for k in _WEIGHT_FIELDS if k in w}      # keep the tensors alive
        ws = CodWeights(*[_ptr(self._weights.get(k)) for k in _WEIGHT_FIELDS])
        _check("cod_set_weights", lib().cod_set_weights(self._h, C.byref(ws), _stream()))

    # ---- the five parts
    def verify_accept(self, draft, target, S, n_forced, state: State, split: Split) -> None:
        st, sp = state.struct(), split.struct()
        _check("cod_verify_accept", lib().cod_verify_accept(self._h, _ptr(draft), _ptr(target), S, n_forced,
                                                            C.byref(st), C.byref(sp), _stream()))

    def project_kv(self, H, split: Split, S, mode, J) -> None:
        sp = split.struct()
        _check("cod_project_kv", lib().cod_project_kv(self._h, _ptr(H), C.byref(sp), S, mode, _ptr(J), _stream()))

    def scatter_kv(self, J, split: Split, S, mode, state: State) -> None:
        st, sp = state.struct(), split.struct()
        _check("cod_scatter_kv", lib().cod_scatter_kv(self._h, _ptr(J), C.byref(sp), S, mode, C.byref(st), _stream()))

    def block_attn(self, layer, q, k_blk, v_blk, state: State, S, use_carry, out, carry_mass=None) -> None:
        st = state.struct()
        _check("cod_block_attn", lib().cod_block_attn(self._h, layer, _ptr(q), _ptr(k_blk), _ptr(v_blk), C.byref(st),
                                                      S, int(use_carry), _ptr(out), _ptr(carry_mass), _stream()))

    def lm_head_argmax(self, x, n_rows, tok, top_logit=None) -> None:
        _check("cod_lm_head_argmax", lib().cod_lm_head_argmax(self._h, _ptr(x), n_rows, _ptr(tok), _ptr(top_logit),
                                                              _stream()))

    def draft_round(self, draft, target, H, S, n_forced, mode, state: State, split: Optional[Split], next_draft,
                    taps: Optional[Taps] = None) -> None:
        st = state.struct()
        sp = split.struct() if split is not None else None
        tp = taps.struct() if taps is not None else None
        _check("cod_draft_round", lib().cod_draft_round(
            self._h, _ptr(draft), _ptr(target), _ptr(H), S, n_forced, mode, C.byref(st),
            C.byref(sp) if sp is not None else None, _ptr(next_draft),
            C.byref(tp) if tp is not None else None, _stream()))

    def verify_accept_stochastic(self, target, p_tok, q_tok, u, S, n_forced, state: State, split: Split) -> None:
        st, sp = state.struct(), split.struct()
        _check("cod_verify_accept_stochastic", lib().cod_verify_accept_stochastic(
            self._h, _ptr(target), _ptr(p_tok), _ptr(q_tok), _ptr(u), S, n_forced, C.byref(st), C.byref(sp), _stream()))

    def draft_round_stochastic(self, target, p_tok, q_tok, u, H, S, n_forced, mode, state: State,
                               split: Optional[Split], next_draft, taps: Optional[Taps] = None,
                               q_next=None, seed: int = 0, step: int = 0) -> None:
        st = state.struct()
        sp = split.struct() if split is not None else None
        tp = taps.struct() if taps is not None else None
        _check("cod_draft_round_stochastic", lib().cod_draft_round_stochastic(
            self._h, _ptr(target), _ptr(p_tok), _ptr(q_tok), _ptr(u), _ptr(H), S, n_forced, mode, C.byref(st),
            C.byref(sp) if sp is not None else None, _ptr(next_draft),
            C.byref(tp) if tp is not None else None, _ptr(q_next), seed, step, _stream()))

    def lm_head_sample(self, x, n_rows, seed, step, tok, q_tok=None, lse=None) -> None:
        _check("cod_lm_head_sample", lib().cod_lm_head_sample(
            self._h, _ptr(x), n_rows, seed, step, _ptr(tok), _ptr(q_tok), _ptr(lse), _stream()))

    def lm_head_rank(self, x, n_rows, ref_tok, rank, ref_logit=None) -> None:
        _check("cod_lm_head_rank", lib().cod_lm_head_rank(
            self._h, _ptr(x), n_rows, _ptr(ref_tok), _ptr(rank), _ptr(ref_logit), _stream()))

    def reconvergence_count(self, z, y, length, S, out) -> None:
        _check("cod_reconvergence_count", lib().cod_reconvergence_count(
            self._h, _ptr(z), _ptr(y), _ptr(length), S, _ptr(out), _stream()))

    # ---- bookkeeping
    def poll_status(self, clear: bool = True) -> int:
        flags = C.c_uint32(0)
        _check("cod_poll_status", lib().cod_poll_status(self._h, C.byref(flags), int(clear), _stream()))
        return int(flags.value)

    def set_wait_limit(self, sm_cycles: int) -> None:
        """Bound of the device-side waits of the weight-streaming contraction, in SM cycles (0: built-in)."""
        _check("cod_set_wait_limit", lib().cod_set_wait_limit(self._h, C.c_longlong(sm_cycles)))

    def selftest_expire_wait(self, on: bool) -> None:
        """While on, that kernel requests no operands: its waits run out and raise COD_DEV_TIMEOUT."""
        _check("cod_selftest_expire_wait", lib().cod_selftest_expire_wait(self._h, int(bool(on))))

    def profile_enable(self, classes=()) -> None:
        mask = 0
        for k in classes:
            mask |= 1 << KERNEL_CLASSES.index(k)
        _check("cod_profile_enable", lib().cod_profile_enable(self._h, mask))

    def profile_read(self, klass: str):
        ms, n = C.c_float(0), C.c_int32(0)
        _check("cod_profile_read", lib().cod_profile_read(self._h, KERNEL_CLASSES.index(klass), C.byref(ms), C.byref(n)))
        return float(ms.value), int(n.value)

    def launch_count(self) -> int:
        return int(lib().cod_launch_count(self._h))

    def workspace_bytes(self) -> int:
        return int(lib().cod_workspace_bytes(self._h))


def lm_head_argmax_static(emb: torch.Tensor, g_final: torch.Tensor, x: torch.Tensor, tok: torch.Tensor,
                          top_logit: Optional[torch.Tensor], rms_eps: float) -> None:
    """cod_lm_head_argmax_static: the LM-head argmax for callers that may not allocate device memory.

    Needs no Context. The scratch is a fixed array inside the library (rows <= 64, width <= 8192);
    calls that overlap on the GPU race on it, and the first call on a device should precede any
    stream capture."""
    n_rows, d_model = x.shape
    dtype = COD_BF16 if emb.dtype == torch.bfloat16 else COD_F32
    _check("cod_lm_head_argmax_static", lib().cod_lm_head_argmax_static(
        _ptr(emb), _ptr(g_final), _ptr(x), n_rows, d_model, emb.shape[0], dtype, C.c_float(rms_eps),
        _ptr(tok), _ptr(top_logit), _stream()))


def make_config(sh, max_batch: int, max_pages_per_seq: int, n_pages: int, attn_split_len: int = 0,
                no_tensor_cores: bool = False, extra_flags: int = 0) -> CodConfig:
    """cod_config from a synthetic DrafterShape."""
    return CodConfig(
        d_target=sh.d_target, n_cap=sh.n_cap, d_model=sh.d_model, n_layers=sh.n_layers, n_q_heads=sh.n_q,
        n_kv_heads=sh.n_kv, head_dim=sh.hd, vocab=sh.vocab, mask_token_id=sh.mask_token_id, block=sh.W,
        page_size=sh.page, max_batch=max_batch, max_pages_per_seq=max_pages_per_seq, n_pages=n_pages,
        dtype=COD_BF16 if sh.dtype == "bf16" else COD_F32,
        flags=extra_flags | (COD_F_HIDDEN_NORM if sh.hidden_norm else 0) | (COD_F_NO_TENSOR_CORES if no_tensor_cores else 0)
        | (COD_F_QK_NORM if sh.qk_norm else 0)
        | {"embedding": 0, "none": COD_F_NO_CARRY_EMBED, "projector": COD_F_REJ_PROJECTOR}[sh.carry_variant],
        rope_theta=sh.rope_theta, rms_eps=sh.rms_eps,
        attn_split_len=attn_split_len, d_ff=sh.d_ff, carry_rounds=sh.carry_rounds)


def weights_to_device(w: Dict[str, np.ndarray], dtype: str) -> Dict[str, torch.Tensor]:
    return {k: to_device(v, dtype) for k, v in w.items()}
