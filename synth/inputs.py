"""Counter-based synthetic Q/K/V for the workloads in `configs.py`.

Every element is a pure function of (seed, tensor kind, sequence, layer, head,
token, dim): a 64-bit integer mix of that counter picks one of 65 536
standard-normal quantiles.  The same torch integer ops run on CPU and on the
GPU, so any slice can be regenerated anywhere and is bit-identical.

Structure on top of the iid N(0,1) field z:
  * per (layer, head) a unit direction u;
  * queries  q = z + sqrt(D) * u        (query mean of norm sqrt(D));
  * keys     k = z + 2 * u  for "planted" visual tokens, k = z otherwise,
    which gives planted tokens a +2 mean logit;
  * values   v = z.
All additions are single fp32 adds of pre-rounded fp32 operands (no fused
multiply-add), then one round-to-nearest-even to the workload dtype.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from .configs import Workload

_GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB

# radices of the element counter (generous fixed bounds, independent of the workload)
_NB, _NL, _NH, _NT, _ND = 64, 64, 64, 8192, 128
_KIND = {"q": 0, "k": 1, "v": 2, "u": 3}


def _i64(c: int) -> int:
    c &= (1 << 64) - 1
    return c - (1 << 64) if c >= (1 << 63) else c


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrapping multiply, logical shifts)."""
    x = x ^ ((x >> 30) & 0x3FFFFFFFF)
    x = x * _i64(_M1)
    x = x ^ ((x >> 27) & 0x1FFFFFFFFF)
    x = x * _i64(_M2)
    x = x ^ ((x >> 31) & 0x1FFFFFFFF)
    return x


_QT_CACHE: dict = {}


def _quantile_table(device) -> torch.Tensor:
    """65 536 standard-normal quantiles, built once on the CPU in fp64, stored as fp32."""
    if "cpu" not in _QT_CACHE:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        _QT_CACHE["cpu"] = torch.special.ndtri(p).to(torch.float32)
    key = str(device)
    if key not in _QT_CACHE:
        _QT_CACHE[key] = _QT_CACHE["cpu"].to(device)
    return _QT_CACHE[key]


def _torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


class SynthInputs:
    """Generator of one workload's tensors, on any device, in any slice."""

    def __init__(self, wl: Workload):
        self.wl = wl
        assert wl.batch <= _NB and wl.num_layers <= _NL and wl.num_heads <= _NH
        assert wl.t0_max + wl.decode_steps + 1 <= _NT and wl.head_dim <= _ND
        rng = np.random.Generator(np.random.PCG64([wl.seed, 0x5151]))
        self.text_len = rng.integers(wl.text_len_min, wl.text_len_max + 1, size=wl.batch).astype(np.int32)
        self._planted = [self._plant(b) for b in range(wl.batch)]
        # unit directions u[l][h][:] (fp64 on the CPU, then fixed fp32 operands)
        zu = self._z("u", [0], range(wl.num_layers), range(wl.num_heads), [0], "cpu")[0, :, :, 0, :].double()
        u = zu / zu.norm(dim=-1, keepdim=True)
        self._u2 = (2.0 * u).to(torch.float32)                          # [L, H, D]
        self._usq = (math.sqrt(wl.head_dim) * u).to(torch.float32)      # [L, H, D]

    # ---------------------------------------------------------------- planted sets
    def _plant(self, b: int):
        wl = self.wl
        rng = np.random.Generator(np.random.PCG64([wl.seed, 0xA11CE, b]))
        nv, npl = wl.num_visual, wl.num_planted
        sets = []
        if wl.planted == "uniform":
            for _ in range(wl.num_layers):
                sets.append(np.sort(rng.choice(nv, size=npl, replace=False)))
        elif wl.planted == "drift":
            cur = list(rng.choice(nv, size=npl, replace=False))
            nrep = max(1, math.ceil(0.10 * npl))
            for _ in range(wl.num_layers):
                sets.append(np.sort(np.array(cur)))
                for j in rng.choice(npl, size=nrep, replace=False):
                    while True:
                        c = int(rng.integers(nv))
                        if c not in cur:
                            cur[j] = c
                            break
        elif wl.planted == "patch":
            g = wl.grid_side
            tiles = nv // (g * g)

            def patch():
                t, r, c = int(rng.integers(tiles)), int(rng.integers(g - 2)), int(rng.integers(g - 2))
                return [t * g * g + (r + i) * g + (c + j) for i in range(3) for j in range(3)]

            npatch = math.ceil(npl / 9)
            patches = [patch() for _ in range(npatch)]
            for _ in range(wl.num_layers):
                flat = []
                for p in patches:
                    for i in p:
                        if i not in flat:
                            flat.append(i)
                sets.append(np.sort(np.array(flat[:npl])))
                patches[int(rng.integers(npatch))] = patch()
        else:
            raise ValueError(wl.planted)
        return sets

    def planted(self, b: int, layer: int) -> np.ndarray:
        """Original visual indices of the planted (attentive) tokens of (b, layer)."""
        return self._planted[b][layer]

    # ---------------------------------------------------------------- the N(0,1) field
    def _z(self, kind, bs, ls, hs, toks, device) -> torch.Tensor:
        """fp32 z[len(bs), len(ls), len(hs), len(toks), D] for the given index lists."""
        wl = self.wl
        dev = torch.device(device)

        def idx(v):
            return torch.as_tensor(list(v) if not torch.is_tensor(v) else v, dtype=torch.int64, device=dev)

        b, l, h, t = idx(bs), idx(ls), idx(hs), idx(toks)
        d = torch.arange(wl.head_dim, dtype=torch.int64, device=dev)
        c = (_KIND[kind] * _NB + b)[:, None] * _NL + l[None, :]               # [b, l]
        c = c[:, :, None] * _NH + h[None, None, :]                            # [b, l, h]
        c = c[:, :, :, None] * _NT + t[None, None, None, :]                   # [b, l, h, t]
        c = c[..., None] * _ND + d                                            # [b, l, h, t, d]
        c = c + _i64(wl.seed * _GOLD + 0x243F6A8885A308D3)
        bits = (_mix64(c) >> 20) & 0xFFFF
        return _quantile_table(dev)[bits]

    # ---------------------------------------------------------------- token indexing
    def gen_token(self, step: int) -> int:
        """Counter index of the token whose k/v is appended at decode step `step` (>= 1)."""
        return self.wl.t0_max + (step - 1)

    def _planted_mask(self, bs, ls, toks, device) -> torch.Tensor:
        """bool [len(bs), len(ls), len(toks)]: prompt token index is a planted visual token."""
        wl = self.wl
        toks = np.asarray(list(toks), dtype=np.int64)
        m = np.zeros((len(bs), len(ls), len(toks)), dtype=bool)
        vis = toks - wl.sys_len
        for i, b in enumerate(bs):
            for j, l in enumerate(ls):
                m[i, j] = np.isin(vis, self._planted[b][l]) & (vis >= 0) & (vis < wl.num_visual)
        return torch.from_numpy(m).to(device)

    # ---------------------------------------------------------------- public tensors
    def kv_rows(self, bs, ls, toks, device="cpu"):
        """K, V [len(bs), len(ls), H, len(toks), D] for arbitrary counter-token indices.

        Prompt token j in [0, t0_max) is system (j < sys), visual (next num_visual) or
        text; `gen_token(step)` gives the index of a generated token.
        """
        wl = self.wl
        bs, ls, toks = list(bs), list(ls), list(toks)
        hs = range(wl.num_heads)
        zk = self._z("k", bs, ls, hs, toks, device)
        zv = self._z("v", bs, ls, hs, toks, device)
        mask = self._planted_mask(bs, ls, toks, device).to(torch.float32)       # [b, l, t]
        u2 = self._u2.to(device)[ls]                                            # [l, H, D]
        shift = mask[:, :, None, :, None] * u2[None, :, :, None, :]
        K = zk + shift
        dt = _torch_dtype(wl.dtype)
        return K.to(dt), zv.to(dt)

    def prompt_kv(self, ls, device="cpu"):
        """K, V [len(ls), B, H, t0_max, D] (rows [S | V | I], padded with zeros past each text length)."""
        wl = self.wl
        ls = list(ls)
        K, V = self.kv_rows(range(wl.batch), ls, range(wl.t0_max), device)
        K, V = K.transpose(0, 1).contiguous(), V.transpose(0, 1).contiguous()
        for b in range(wl.batch):
            t0 = wl.sys_len + wl.num_visual + int(self.text_len[b])
            K[:, b, :, t0:] = 0
            V[:, b, :, t0:] = 0
        return K, V

    def queries(self, steps, ls=None, device="cpu"):
        """q [len(steps), len(ls), B, H, D]; step 0 is the last prompt token's query."""
        wl = self.wl
        ls = list(range(wl.num_layers)) if ls is None else list(ls)
        z = self._z("q", range(wl.batch), ls, range(wl.num_heads), list(steps), device)   # [B, l, H, s, D]
        q = z + self._usq.to(device)[ls][None, :, :, None, :]
        return q.permute(3, 1, 0, 2, 4).contiguous().to(_torch_dtype(wl.dtype))

    def new_kv(self, steps, ls=None, device="cpu"):
        """k_new, v_new [len(steps), len(ls), B, H, D] of the tokens appended at decode steps >= 1."""
        wl = self.wl
        ls = list(range(wl.num_layers)) if ls is None else list(ls)
        toks = [self.gen_token(s) for s in steps]
        K, V = self.kv_rows(range(wl.batch), ls, toks, device)                            # [B, l, H, s, D]
        return K.permute(3, 1, 0, 2, 4).contiguous(), V.permute(3, 1, 0, 2, 4).contiguous()
