"""Runs the CUDA library and the CPU oracle side by side on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import cod_oracle as orc
from paper_2609_14717_b200 import binding as B
from paper_2609_14717_b200 import synth
from tests.helpers import oracle_config

TOL = {"bf16": 2e-2, "f32": 1e-3}      # max |gpu - ref| / max |ref| per tensor
GAP = 1e-2                             # argmax must agree where the oracle's top-2 gap is at least this


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


class Pair:
    """One workload instantiated on both sides with identical weights, layout and pool."""

    def __init__(self, wl: synth.Workload, seed: int, attn_split_len: int = 0, wo_scale: float = 1.0,
                 fill_pool: bool = True, max_batch: int | None = None, poison: bool = False, extra_flags: int = 0):
        self.wl, self.seed = wl, seed
        sh = wl.shape
        self.cfg_o = oracle_config(sh)
        lay = synth.make_layout(wl, seed)
        self.lay = lay
        n_pages, mp = int(lay["n_pages"]), int(lay["max_pages_per_seq"])
        w = synth.make_weights(sh, seed)
        if wo_scale != 1.0:
            w["wo"] = synth.to_storage(w["wo"] * np.float32(wo_scale), sh.dtype)
        self.w_host = w
        self.w_o = orc.prepare_weights(w)
        self.st_o = orc.OracleState(self.cfg_o, wl.S, n_pages, lay["block_table"], lay["committed_len"])
        self.cfg_g = B.make_config(sh, max_batch or wl.S, mp, n_pages, attn_split_len, extra_flags=extra_flags)
        self.ctx = B.Context(self.cfg_g)
        self.w_g = B.weights_to_device(w, sh.dtype)
        self.ctx.set_weights(self.w_g)
        self.st_g = B.State(self.cfg_g, sh.dtype, wl.S, lay["block_table"], lay["committed_len"])
        if poison:
            self.st_g.kv_pool.fill_(float("nan"))
            self.st_g.carry_kv.fill_(float("nan"))
            self.st_o.pool[:] = np.nan
        if fill_pool:
            for l in range(sh.n_layers):
                pl = synth.pool_layer(wl, seed, l, n_pages)
                if poison:
                    # only the pages a sequence has committed rows in are defined
                    keep = np.zeros(n_pages, dtype=bool)
                    for s in range(wl.S):
                        used = (int(lay["committed_len"][s]) + sh.page - 1) // sh.page
                        keep[lay["block_table"][s, :used]] = True
                    pl[~keep] = np.nan
                    for s in range(wl.S):                      # rows past L in the last, partial page
                        Ls = int(lay["committed_len"][s])
                        if Ls % sh.page:
                            pl[lay["block_table"][s, Ls // sh.page], :, :, Ls % sh.page:, :] = np.nan
                self.st_o.pool[l] = pl
                self.st_g.kv_pool[l] = B.to_device(pl, sh.dtype)
        self.split = B.Split(wl.S, sh.W)
        self.taps = B.Taps(self.cfg_g, wl.S)
        self.next_draft = torch.zeros((wl.S, sh.W), dtype=torch.int32, device="cuda")

    def round_inputs(self, r: int):
        rd = synth.make_round(self.wl, self.seed, r)
        dev = {"draft": dev_i32(rd["draft"]), "target": dev_i32(rd["target"]),
               "H": B.to_device(rd["H"], self.wl.shape.dtype)}
        return rd, dev

    def run_round(self, r: int, mode: int, n_forced: int | None = None, rd=None, dev=None):
        wl = self.wl
        if rd is None:
            rd, dev = self.round_inputs(r)
        nf = wl.n_forced if n_forced is None else n_forced
        res_o = orc.draft_round(rd["draft"], rd["target"], rd["H"], self.st_o, self.w_o, nf, mode)
        self.ctx.draft_round(dev["draft"], dev["target"], dev["H"], wl.S, nf, mode, self.st_g, self.split,
                             self.next_draft, self.taps)
        torch.cuda.synchronize()
        return res_o

    # ---- comparisons
    def check_split(self, res_o):
        got = self.split.to_host()
        for k, v in res_o["split"].items():
            assert np.array_equal(got[k], v), f"split.{k} differs"

    def check_lens(self):
        assert np.array_equal(self.st_g.committed_len.cpu().numpy(), self.st_o.committed_len)
        assert np.array_equal(self.st_g.carry_len.cpu().numpy(), self.st_o.carry_len)

    def written_kv_errors(self, res_o, L_before):
        """Relative error of the K/V rows this round wrote (committed slots and carry rows)."""
        wl, sh = self.wl, self.wl.shape
        pool_g = self.st_g.kv_pool.float().cpu().numpy().astype(np.float64)
        carry_g = self.st_g.carry_kv.float().cpu().numpy().astype(np.float64)
        m = res_o["split"]["accept_len"]
        errs = []
        for l in range(sh.n_layers):
            ref, got = [], []
            for s in range(wl.S):
                for p in range(int(m[s])):
                    pos = int(L_before[s]) + p
                    pg, off = int(self.st_o.block_table[s, pos // sh.page]), pos % sh.page
                    ref.append(self.st_o.pool[l, pg, :, :, off, :]); got.append(pool_g[l, pg, :, :, off, :])
                c = int(self.st_o.carry_len[s])
                if c:
                    ref.append(self.st_o.carry[l, s, :, :, :c, :].reshape(-1, sh.hd))
                    got.append(carry_g[l, s, :, :, :c, :].reshape(-1, sh.hd))
            if ref:
                ref = np.concatenate([a.reshape(-1) for a in ref]); got = np.concatenate([a.reshape(-1) for a in got])
                errs.append(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))
        return errs

    def close(self):
        self.ctx.close()
