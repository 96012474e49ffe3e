"""Seeded synthetic logits for the GTO draft-tree pass.

Input generators only: nothing of the method's arithmetic lives here.  Both the CUDA
path and the CPU oracle consume the tensors this module makes (the oracle reads the
generated values back from wherever they were generated, so device differences in
log / cos cannot affect parity).

Every value is a pure function of (seed, stream, absolute element index): a
splitmix64-style counter hash gives two 24-bit uniforms, Box-Muller turns them into
a normal.  The index uses the absolute position number b, so a sub-batch or a shard
of positions sees the same rows as the full batch.

The synthetic rows stand in for the logits a drafter / target pair would emit on
training prefixes; the shapes are those of the models named in each workload.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np
import torch

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the signed value torch.int64 holds for those bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _s64(0x9E3779B97F4A7C15)
_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrap-around arithmetic)."""
    x = x + _GOLD
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _mix64_int(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & _M64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _M64
    return x ^ (x >> 31)


def stream_key(seed: int, *parts: int) -> int:
    """Key of a sub-stream: chained hash of the seed and small integers."""
    h = _mix64_int(seed)
    for p in parts:
        h = _mix64_int(h ^ (p & _M64))
    return h


def _bits(counter: torch.Tensor, key: int) -> torch.Tensor:
    return _mix64(_mix64(counter ^ _s64(key)))


def uniforms(counter: torch.Tensor, key: int):
    """Two fp32 uniforms per counter: u1 in (0, 1], u2 in [0, 1)."""
    h = _bits(counter, key)
    u1 = ((_lsr(h, 40) & 0xFFFFFF) + 1).to(torch.float32) * (1.0 / 16777216.0)
    u2 = (_lsr(h, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)
    return u1, u2


def normals(counter: torch.Tensor, key: int) -> torch.Tensor:
    """One fp32 standard normal per counter (Box-Muller)."""
    u1, u2 = uniforms(counter, key)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def hash_normal(seed: int, row, token) -> np.ndarray:
    """fp64 standard normal as a pure function of (seed, row, token); numpy, host.

    Used for the old-policy perturbation: old_logp = path_logp + 0.05 * hash_normal.
    """
    row = np.asarray(row, dtype=np.int64)
    token = np.asarray(token, dtype=np.int64)
    out = np.empty(np.broadcast(row, token).shape, dtype=np.float64)
    rb, tb = np.broadcast_arrays(row, token)
    for idx in np.ndindex(out.shape):
        h = _mix64_int(stream_key(seed, 0x0FD, int(rb[idx]), int(tb[idx])))
        u1 = (((h >> 40) & 0xFFFFFF) + 1) / 16777216.0
        u2 = ((h >> 16) & 0xFFFFFF) / 16777216.0
        out[idx] = math.sqrt(-2.0 * math.log(u1)) * math.cos(2.0 * math.pi * u2)
    return out


# ------------------------------------------------------------------ workloads
@dataclass(frozen=True)
class Workload:
    """Shape and value recipe of one synthetic workload."""
    name: str
    B: int
    V_draft: int
    V_target: int
    D: int
    k: int
    g: int
    G: int = 2
    m: int = 8
    dtype: str = "bf16"          # "bf16", "f16" or "f32"
    sigma_t: float = 2.5         # scale of the target base distribution
    boost: float = 8.0           # added to the seeded true token of every target row
    sigma_d: float = 0.7         # draft = target + N(0, sigma_d^2)
    student_t: bool = False      # target base ~ Student-t(4) instead of normal
    seed: int = 0
    eta: float = 1.0
    clip_eps: float = 0.2
    std_delta: float = 1e-6
    grad_scale: float = 1.0
    old_sigma: float = 0.05

    @property
    def R(self) -> int:
        return 1 + (self.D - 1) * self.k

    @property
    def P(self) -> int:
        return self.k + (self.D - 1) * self.k * self.k

    @property
    def torch_dtype(self):
        return {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def with_B(self, B: int) -> "Workload":
        return replace(self, B=B)


def _seed(i: int) -> int:
    return 250922134 * 16 + i


WORKLOADS = {
    0: Workload("tiny", B=8, V_draft=512, V_target=512, D=3, k=4, g=12, dtype="f32", seed=_seed(0)),
    1: Workload("vicuna-1.3-13b-shape", B=512, V_draft=32000, V_target=32000, D=6, k=10, g=60,
                seed=_seed(1)),
    2: Workload("llama-3.1-8b-shape", B=1024, V_draft=32000, V_target=128256, D=7, k=10, g=60,
                seed=_seed(2)),
    3: Workload("qwen3-8b-shape", B=512, V_draft=151936, V_target=151936, D=7, k=10, g=60,
                sigma_t=3.0, boost=7.0, sigma_d=0.9, student_t=True, seed=_seed(3)),
    4: Workload("llama-3.3-70b-shape", B=2048, V_draft=32000, V_target=128256, D=8, k=10, g=60,
                seed=_seed(4)),
}

_S_TARGET, _S_CHI, _S_TRUE, _S_DRAFT, _S_D2T = 1, 2, 3, 4, 5


def make_d2t(w: Workload) -> torch.Tensor | None:
    """Injective, increasing draft-id -> target-id map (None when the vocabularies
    coincide): the V_draft ids with the smallest hash out of V_target, sorted."""
    if w.V_draft == w.V_target:
        return None
    ids = torch.arange(w.V_target, dtype=torch.int64)
    score = _lsr(_bits(ids, stream_key(w.seed, _S_D2T)), 1)
    keep = torch.argsort(score, stable=True)[: w.V_draft]
    return torch.sort(keep).values.to(torch.int32)


def _target_base(w: Workload, b0: int, nb: int, device, d2t_dev) -> torch.Tensor:
    """fp32 target logits [nb, R, V_target] of positions b0 .. b0+nb-1."""
    R, Vt = w.R, w.V_target
    row = (torch.arange(b0, b0 + nb, device=device, dtype=torch.int64)[:, None] * R
           + torch.arange(R, device=device, dtype=torch.int64)[None, :])            # [nb, R]
    cnt = row[:, :, None] * Vt + torch.arange(Vt, device=device, dtype=torch.int64)  # [nb,R,Vt]
    z = normals(cnt, stream_key(w.seed, _S_TARGET))
    if w.student_t:
        u1, u2 = uniforms(cnt, stream_key(w.seed, _S_CHI))
        chi2 = -2.0 * torch.log(u1 * (1.0 - u2))          # chi-square, 4 degrees of freedom
        z = z / torch.sqrt(chi2 / 4.0)
    del cnt
    z = z * w.sigma_t
    h = _lsr(_bits(row, stream_key(w.seed, _S_TRUE)), 1)
    if d2t_dev is None:
        true_tok = h % Vt
    else:
        true_tok = d2t_dev.to(torch.int64)[h % w.V_draft]
    z.scatter_add_(2, true_tok[:, :, None], torch.full_like(true_tok, w.boost, dtype=torch.float32)[:, :, None])
    return z


def generate(w: Workload, device="cpu", b0: int = 0, chunk_elems: int = 1 << 25):
    """Materialise the workload's tensors for positions b0 .. b0+B-1 on `device`.

    Returns dict(draft [G,B,D,k,V_draft], target [G,B,R,V_target], d2t [V_draft] int32
    or None).  Target rows: sigma_t * base noise, + boost on one seeded true token
    per row (drawn from the mapped ids when the draft vocabulary is reduced); both
    trees see the same target rows.  Draft rows: the target row restricted to the
    mapped ids plus an independent N(0, sigma_d^2) draw per tree.  The unused draft
    rows [.,.,0,1:,:] are filled with NaN so that a read of them is noticed.
    """
    G, B, D, k, R = w.G, w.B, w.D, w.k, w.R
    Vd, Vt = w.V_draft, w.V_target
    dt = w.torch_dtype
    d2t = make_d2t(w)
    d2t_dev = None if d2t is None else d2t.to(device)
    draft = torch.empty((G, B, D, k, Vd), dtype=dt, device=device)
    target = torch.empty((G, B, R, Vt), dtype=dt, device=device)
    draft[:, :, 0, 1:, :] = float("nan")
    dview = draft.view(G, B, D * k, Vd)
    nb_max = max(1, chunk_elems // (R * Vt))
    for c0 in range(0, B, nb_max):
        nb = min(nb_max, B - c0)
        zt = _target_base(w, b0 + c0, nb, device, d2t_dev)            # [nb,R,Vt] fp32
        zt_store = zt.to(dt)
        for t in range(G):
            target[t, c0:c0 + nb] = zt_store
        base = zt if d2t_dev is None else zt.index_select(2, d2t_dev.to(torch.int64))
        del zt
        row = (torch.arange(b0 + c0, b0 + c0 + nb, device=device, dtype=torch.int64)[:, None] * R
               + torch.arange(R, device=device, dtype=torch.int64)[None, :])
        cnt = row[:, :, None] * Vd + torch.arange(Vd, device=device, dtype=torch.int64)
        for t in range(G):
            zd = (base + w.sigma_d * normals(cnt, stream_key(w.seed, _S_DRAFT, t))).to(dt)
            dview[t, c0:c0 + nb, 0] = zd[:, 0]
            if R > 1:
                dview[t, c0:c0 + nb, k:] = zd[:, 1:]
            del zd
        del base, cnt
    return dict(draft=draft, target=target, d2t=d2t_dev)


def old_logp_from_path(w: Workload, path_logp: np.ndarray, path_row: np.ndarray,
                       path_token: np.ndarray, path_len: np.ndarray, b0: int = 0) -> np.ndarray:
    """Old-policy log-probabilities of the accepted path: the current ones plus
    old_sigma * hash_normal(seed, global draft row, token).  Host, fp64; entries
    beyond path_len are 0."""
    B, D = path_logp.shape
    out = np.zeros((B, D), dtype=np.float64)
    for b in range(B):
        for j in range(int(path_len[b])):
            grow = (b0 + b) * w.R + int(path_row[b, j])
            out[b, j] = float(path_logp[b, j]) + w.old_sigma * float(
                hash_normal(w.seed, grow, int(path_token[b, j])))
    return out
