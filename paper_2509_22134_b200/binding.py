"""ctypes binding of libgto.so: argument marshalling only.

The functions carry the names of the C entry points (include/gto.h) and take torch
tensors for device buffers; PyTorch supplies device memory and streams, every step of
the pass runs in the library's kernels.  Importing this module loads the library and
raises if it has not been built - there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgto.so")

GTO_OK = 0
GTO_F32, GTO_BF16, GTO_F16 = 0, 1, 2
GTO_AGG_LSE, GTO_AGG_MAX, GTO_AGG_MEAN = 0, 1, 2
GTO_FLAG_STD_UNBIASED, GTO_FLAG_NO_DEBIAS, GTO_FLAG_GRAD_LIVE_ROWS, GTO_FLAG_SEQ_ALL_NODES = 1, 2, 4, 8
GTO_FLAG_FORCE_ROW_SPLIT = 16
GTO_FLAG_PATH_MAX_EXPECTED = 32

if not os.path.exists(LIB_PATH):
    raise RuntimeError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2509_22134_b200.build` "
        "(the GTO pass has no CPU or PyTorch fallback)")
_lib = ctypes.CDLL(LIB_PATH)


class gto_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "G", "D", "k", "g", "m", "V_draft", "V_target", "logit_dtype", "reward_agg")] + \
               [(n, ctypes.c_float) for n in ("eta", "clip_eps", "std_delta", "grad_scale")] + \
               [("flags", ctypes.c_uint32)]


_TREE_FIELDS = [("node_token", torch.int32), ("node_parent", torch.int32), ("node_depth", torch.int32),
                ("node_ctx_row", torch.int32), ("node_slot", torch.int32), ("node_pool", torch.int32),
                ("node_logp", torch.float32), ("node_score", torch.float64),
                ("node_mask", torch.int64), ("row_lse", torch.float64)]
_REWARD_FIELDS = [("reward", torch.float64), ("etree", torch.float64), ("n_leaves", torch.int32),
                  ("node_ptarget", torch.float32), ("node_pathprod", torch.float32),
                  ("node_L", torch.float32), ("row_lse_t", torch.float64),
                  ("row_argmax_t", torch.int32), ("path_len", torch.int32),
                  ("path_node", torch.int32), ("path_row", torch.int32),
                  ("path_token", torch.int32), ("path_logp", torch.float32)]
_TOKEN_FIELDS = [("loss", torch.float64), ("lse_t", torch.float64)]
_STATS_FIELDS = [("R", torch.float64), ("adv", torch.float64), ("ratio", torch.float64),
                 ("coeff", torch.float64), ("active", torch.int32), ("loss", torch.float64)]


def _struct(name, fields):
    return type(name, (ctypes.Structure,), {"_fields_": [(n, ctypes.c_void_p) for n, _ in fields]})


gto_tree = _struct("gto_tree", _TREE_FIELDS)
gto_reward = _struct("gto_reward", _REWARD_FIELDS)
gto_grad_stats = _struct("gto_grad_stats", _STATS_FIELDS)
gto_token_stats = _struct("gto_token_stats", _TOKEN_FIELDS)

_vp = ctypes.c_void_p
_lib.gto_create.argtypes = [ctypes.POINTER(_vp), ctypes.POINTER(gto_config), ctypes.c_int]
_lib.gto_destroy.argtypes = [_vp]
_lib.gto_build_tree.argtypes = [_vp, _vp, ctypes.POINTER(gto_tree), _vp]
_lib.gto_build_tree_noalloc.argtypes = [ctypes.POINTER(gto_config), ctypes.c_int, _vp,
                                        ctypes.POINTER(gto_tree), _vp]
_lib.gto_build_tree_noalloc.restype = ctypes.c_int
_lib.gto_tree_reward.argtypes = [_vp, ctypes.POINTER(gto_tree), _vp, _vp, ctypes.POINTER(gto_reward), _vp]
_lib.gto_tree_reward_host.argtypes = [_vp, ctypes.POINTER(gto_tree), _vp, _vp, _vp,
                                      ctypes.POINTER(gto_reward), _vp, ctypes.POINTER(ctypes.c_int64)]
_lib.gto_tree_reward_host.restype = ctypes.c_int
_lib.gto_group_surrogate_grad.argtypes = [_vp, _vp, ctypes.POINTER(gto_tree), ctypes.POINTER(gto_reward),
                                          _vp, _vp, ctypes.POINTER(gto_grad_stats), _vp]
_lib.gto_token_loss.argtypes = [_vp, _vp, _vp, _vp, ctypes.POINTER(gto_tree), ctypes.c_float, _vp,
                                ctypes.POINTER(gto_token_stats), _vp]
_lib.gto_token_loss.restype = ctypes.c_int
_lib.gto_token_loss_accumulate.argtypes = [_vp, _vp, _vp, _vp, ctypes.POINTER(gto_tree),
                                           ctypes.POINTER(gto_reward), ctypes.POINTER(gto_grad_stats),
                                           ctypes.c_float, _vp, ctypes.POINTER(gto_token_stats), _vp]
_lib.gto_token_loss_accumulate.restype = ctypes.c_int
_lib.gto_sample_groups.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                   ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int32)]
_lib.gto_sample_groups.restype = ctypes.c_int
_lib.gto_device_status.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_int32)]
_lib.gto_launch_count.argtypes = [_vp]
_lib.gto_launch_count.restype = ctypes.c_int64
_lib.gto_kernel_timing.argtypes = [_vp, ctypes.c_int]
_lib.gto_kernel_times.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
_lib.gto_status_string.argtypes = [ctypes.c_int]
_lib.gto_status_string.restype = ctypes.c_char_p
for _f in ("gto_create", "gto_destroy", "gto_build_tree", "gto_tree_reward",
           "gto_group_surrogate_grad", "gto_device_status", "gto_kernel_timing", "gto_kernel_times"):
    getattr(_lib, _f).restype = ctypes.c_int


class GtoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {gto_status_string(code)} (status {code})")


def gto_status_string(code: int) -> str:
    return _lib.gto_status_string(code).decode()


def _check(code: int, where: str):
    if code != GTO_OK:
        raise GtoError(code, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _fill(struct_type, fields, bufs: dict):
    s = struct_type()
    for name, dtype in fields:
        t = bufs[name]
        assert t.is_cuda and t.is_contiguous() and t.dtype == dtype, name
        setattr(s, name, t.data_ptr())
    return s


def make_config(B, D, k, g, m, V_draft, V_target, dtype, G=2, eta=1.0, clip_eps=0.2,
                std_delta=1e-6, grad_scale=1.0, reward_agg=GTO_AGG_LSE, flags=0) -> gto_config:
    code = {torch.bfloat16: GTO_BF16, torch.float32: GTO_F32, torch.float16: GTO_F16,
            "bf16": GTO_BF16, "f32": GTO_F32, "f16": GTO_F16}[dtype]
    return gto_config(B, G, D, k, g, m, V_draft, V_target, code, reward_agg,
                      eta, clip_eps, std_delta, grad_scale, flags)


def gto_create(cfg: gto_config, device: int = 0) -> int:
    h = _vp()
    _check(_lib.gto_create(ctypes.byref(h), ctypes.byref(cfg), device), "gto_create")
    return h.value


def gto_destroy(ctx: int):
    _check(_lib.gto_destroy(ctx), "gto_destroy")


def alloc_tree(cfg: gto_config, device) -> dict:
    G, B, g, R = cfg.G, cfg.B, cfg.g, 1 + (cfg.D - 1) * cfg.k
    W = (g + 63) // 64
    shapes = {"node_mask": (G, B, g, W), "row_lse": (G, B, R)}
    return {n: torch.empty(shapes.get(n, (G, B, g)), dtype=dt, device=device) for n, dt in _TREE_FIELDS}


def alloc_reward(cfg: gto_config, device) -> dict:
    G, B, g, D, R = cfg.G, cfg.B, cfg.g, cfg.D, 1 + (cfg.D - 1) * cfg.k
    shapes = {"reward": (G, B), "etree": (G, B), "n_leaves": (G, B), "row_lse_t": (G, B, R),
              "row_argmax_t": (G, B, R), "path_len": (B,), "path_node": (B, D), "path_row": (B, D),
              "path_token": (B, D), "path_logp": (B, D)}
    return {n: torch.empty(shapes.get(n, (G, B, g)), dtype=dt, device=device) for n, dt in _REWARD_FIELDS}


def alloc_grad_stats(cfg: gto_config, device) -> dict:
    B = cfg.B
    return {n: torch.empty((B // cfg.m,) if n == "loss" else (B,), dtype=dt, device=device)
            for n, dt in _STATS_FIELDS}


def gto_build_tree(ctx: int, draft: torch.Tensor, tree: dict, stream=None):
    assert draft.is_cuda and draft.is_contiguous()
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    _check(_lib.gto_build_tree(ctx, draft.data_ptr(), ctypes.byref(t), _stream_ptr(stream)),
           "gto_build_tree")


GTO_NOALLOC_MAX_ENTRIES = 1 << 20


def gto_build_tree_noalloc(cfg: gto_config, device: int, draft: torch.Tensor, tree: dict, stream=None):
    """gto_build_tree without a context and without any device allocation: for callers
    that must keep every device byte under their own allocator.  Raises GtoError(7) when
    G*B*R*k exceeds GTO_NOALLOC_MAX_ENTRIES."""
    assert draft.is_cuda and draft.is_contiguous()
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    _check(_lib.gto_build_tree_noalloc(ctypes.byref(cfg), device, draft.data_ptr(), ctypes.byref(t),
                                       _stream_ptr(stream)), "gto_build_tree_noalloc")


def gto_tree_reward(ctx: int, tree: dict, target: torch.Tensor, d2t, reward: dict, stream=None):
    assert target.is_cuda and target.is_contiguous()
    if d2t is not None:
        assert d2t.is_cuda and d2t.dtype == torch.int32 and d2t.is_contiguous()
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    r = _fill(gto_reward, _REWARD_FIELDS, reward)
    _check(_lib.gto_tree_reward(ctx, ctypes.byref(t), target.data_ptr(),
                                None if d2t is None else d2t.data_ptr(), ctypes.byref(r),
                                _stream_ptr(stream)), "gto_tree_reward")


def gto_tree_reward_host(ctx: int, tree: dict, target_host: torch.Tensor, target_dev: torch.Tensor,
                         d2t, reward: dict, stream=None) -> int:
    """gto_tree_reward with the target logits in (pinned) host memory: copies only the
    needed rows into target_dev.  Returns the number of rows copied."""
    assert not target_host.is_cuda and target_host.is_contiguous()
    assert target_dev.is_cuda and target_dev.is_contiguous()
    assert target_host.shape == target_dev.shape and target_host.dtype == target_dev.dtype
    if d2t is not None:
        assert d2t.is_cuda and d2t.dtype == torch.int32 and d2t.is_contiguous()
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    r = _fill(gto_reward, _REWARD_FIELDS, reward)
    n = ctypes.c_int64(0)
    _check(_lib.gto_tree_reward_host(ctx, ctypes.byref(t), target_host.data_ptr(), target_dev.data_ptr(),
                                     None if d2t is None else d2t.data_ptr(), ctypes.byref(r),
                                     _stream_ptr(stream), ctypes.byref(n)), "gto_tree_reward_host")
    return int(n.value)


def gto_group_surrogate_grad(ctx: int, draft: torch.Tensor, tree: dict, reward: dict,
                             old_logp: torch.Tensor, grad: torch.Tensor, stats: dict, stream=None):
    assert old_logp.is_cuda and old_logp.dtype == torch.float32 and old_logp.is_contiguous()
    assert grad.is_cuda and grad.is_contiguous() and grad.dtype == draft.dtype
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    r = _fill(gto_reward, _REWARD_FIELDS, reward)
    s = _fill(gto_grad_stats, _STATS_FIELDS, stats)
    _check(_lib.gto_group_surrogate_grad(ctx, draft.data_ptr(), ctypes.byref(t), ctypes.byref(r),
                                         old_logp.data_ptr(), grad.data_ptr(), ctypes.byref(s),
                                         _stream_ptr(stream)), "gto_group_surrogate_grad")


def alloc_token_stats(cfg: gto_config, device) -> dict:
    return {n: torch.empty((cfg.B,), dtype=dt, device=device) for n, dt in _TOKEN_FIELDS}


def gto_token_loss(ctx: int, draft: torch.Tensor, target: torch.Tensor, d2t, tree: dict, weight: float,
                   grad_root: torch.Tensor, stats: dict, stream=None):
    assert draft.is_cuda and draft.is_contiguous() and target.is_cuda and target.is_contiguous()
    assert grad_root.is_cuda and grad_root.is_contiguous() and grad_root.dtype == draft.dtype
    if d2t is not None:
        assert d2t.is_cuda and d2t.dtype == torch.int32 and d2t.is_contiguous()
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    s = _fill(gto_token_stats, _TOKEN_FIELDS, stats)
    _check(_lib.gto_token_loss(ctx, draft.data_ptr(), target.data_ptr(),
                               None if d2t is None else d2t.data_ptr(), ctypes.byref(t),
                               ctypes.c_float(weight), grad_root.data_ptr(), ctypes.byref(s),
                               _stream_ptr(stream)), "gto_token_loss")


def gto_token_loss_accumulate(ctx: int, draft: torch.Tensor, target: torch.Tensor, d2t, tree: dict,
                              reward: dict, stats: dict, weight: float, grad: torch.Tensor,
                              token_stats: dict, stream=None):
    """gto_token_loss into slice [b, 0, :] of the surrogate's gradient buffer [B, D, V_draft]."""
    assert draft.is_cuda and draft.is_contiguous() and target.is_cuda and target.is_contiguous()
    assert grad.is_cuda and grad.is_contiguous() and grad.dtype == draft.dtype and grad.dim() == 3
    if d2t is not None:
        assert d2t.is_cuda and d2t.dtype == torch.int32 and d2t.is_contiguous()
    t = _fill(gto_tree, _TREE_FIELDS, tree)
    r = _fill(gto_reward, _REWARD_FIELDS, reward)
    g = _fill(gto_grad_stats, _STATS_FIELDS, stats)
    s = _fill(gto_token_stats, _TOKEN_FIELDS, token_stats)
    _check(_lib.gto_token_loss_accumulate(ctx, draft.data_ptr(), target.data_ptr(),
                                          None if d2t is None else d2t.data_ptr(), ctypes.byref(t),
                                          ctypes.byref(r), ctypes.byref(g), ctypes.c_float(weight),
                                          grad.data_ptr(), ctypes.byref(s), _stream_ptr(stream)),
           "gto_token_loss_accumulate")


def gto_sample_groups(s: int, m: int, K: int, u) -> list:
    """Start indices (1-based) of K non-overlapping groups of m adjacent positions (host only)."""
    uu = (ctypes.c_double * max(K, 1))(*[float(x) for x in list(u)[:K]])
    out = (ctypes.c_int32 * max(K, 1))()
    _check(_lib.gto_sample_groups(s, m, K, uu, out), "gto_sample_groups")
    return [int(out[i]) for i in range(K)]


def gto_device_status(ctx: int, stream=None) -> int:
    code = ctypes.c_int32(0)
    _check(_lib.gto_device_status(ctx, _stream_ptr(stream), ctypes.byref(code)), "gto_device_status")
    return code.value


def gto_launch_count(ctx: int) -> int:
    return int(_lib.gto_launch_count(ctx))


KERNEL_NAMES = ["draft_rows", "tree_build", "reward_plan", "target_rows", "tree_reward",
                "group_stats", "grad_rows", "token_loss"]   # GTO_K_* order


def gto_kernel_timing(ctx: int, enable: bool):
    _check(_lib.gto_kernel_timing(ctx, int(bool(enable))), "gto_kernel_timing")


def gto_kernel_times(ctx: int, stream=None) -> dict:
    """{kernel name: (total device ms, launches)} since the last call; synchronises."""
    n = len(KERNEL_NAMES)
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_int64 * n)()
    _check(_lib.gto_kernel_times(ctx, _stream_ptr(stream), ms, cnt), "gto_kernel_times")
    return {name: (ms[i], cnt[i]) for i, name in enumerate(KERNEL_NAMES)}


EXPORTS = ["gto_create", "gto_destroy", "gto_build_tree", "gto_tree_reward",
           "gto_group_surrogate_grad", "gto_device_status", "gto_launch_count", "gto_status_string",
           "gto_kernel_timing", "gto_kernel_times", "gto_build_tree_noalloc", "gto_token_loss", "gto_sample_groups", "gto_tree_reward_host",
           "gto_token_loss_accumulate"]
