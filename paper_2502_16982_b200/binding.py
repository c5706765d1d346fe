"""ctypes binding of the Muon C ABI (include/muon.h).

Argument marshalling only: every step of the optimizer runs in the CUDA
kernels of libmuon_b200.so.  PyTorch supplies device memory and streams.
The functions carry the C names; :class:`MuonContext` bundles them for the
usual init / step / status / destroy life cycle.
"""

from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmuon_b200.so")

MUON_OK = 0
MUON_ERR_INVALID_ARG = -1
MUON_ERR_UNSUPPORTED = -2
MUON_ERR_ALIGNMENT = -3
MUON_ERR_WORKSPACE = -4
MUON_ERR_CUDA = -5
MUON_ERR_TIMEOUT = -6
MUON_ERR_NONFINITE = -7
MUON_DTYPE_BF16 = 0
MUON_DTYPE_FP32 = 1
MUON_TAP_X0, MUON_TAP_A, MUON_TAP_B, MUON_TAP_X = 0, 1, 2, 3
MUON_SCALE_ADJUSTED_LR, MUON_SCALE_FIXED_DIM, MUON_SCALE_UPDATE_NORM = 0, 1, 2

EXPORTED = [
    "muon_workspace_bytes", "muon_partition", "muon_partition_slots", "muon_plan_buckets", "muon_plan_flops", "muon_plan_work", "muon_debug_tile_table", "muon_init", "muon_step", "muon_step_bucket",
    "muon_step_host", "muon_status",
    "muon_get_norms", "muon_get_update_rms", "muon_destroy", "muon_last_error", "muon_last_launch_count",
    "muon_debug_keep", "muon_debug_read", "muon_debug_set_chunk_bytes", "muon_debug_set_pair_fold", "muon_debug_set_tile_mode",
    "muon_debug_wait_expiry",
    "muon_profile_enable", "muon_profile_read", "muon_debug_tmem_bases",
    "muon_momentum_norm_static", "muon_adamw_step",
]
MUON_STATIC_MAX_TILES = 65536
KERNEL_KINDS = ["momentum", "norm", "gram", "poly", "comb", "update"]


class muon_group(C.Structure):
    _fields_ = [
        ("rows", C.c_int32), ("cols", C.c_int32), ("count", C.c_int32),
        ("w_dtype", C.c_int32), ("g_dtype", C.c_int32), ("reserved", C.c_int32),
        ("w", C.POINTER(C.c_void_p)), ("g", C.POINTER(C.c_void_p)), ("m", C.POINTER(C.c_void_p)),
        ("ld_w", C.c_int64), ("ld_g", C.c_int64), ("ld_m", C.c_int64),
        ("w_shadow", C.POINTER(C.c_void_p)), ("ld_shadow", C.c_int64),
    ]


class muon_hparams(C.Structure):
    _fields_ = [
        ("lr", C.c_float), ("wd", C.c_float), ("mu", C.c_float),
        ("nesterov", C.c_int32), ("ns_steps", C.c_int32),
        ("a", C.c_float), ("b", C.c_float), ("c", C.c_float),
        ("eps", C.c_float), ("rms_scale", C.c_float),
        ("scale_mode", C.c_int32), ("scale_dim", C.c_float),
        ("coeffs", C.POINTER(C.c_float)), ("protect_momentum", C.c_int32),
    ]


class muon_adamw_tensor(C.Structure):
    _fields_ = [("p", C.c_void_p), ("g", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p),
                ("numel", C.c_int64), ("p_dtype", C.c_int32), ("g_dtype", C.c_int32)]


class muon_adamw_hparams(C.Structure):
    _fields_ = [("lr", C.c_float), ("wd", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("step", C.c_int32)]


class MuonError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("muon error %d: %s" % (code, msg))
        self.code = code


_lib = None


def lib():
    """Load libmuon_b200.so (once).  There is no fallback: a missing library
    is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libmuon_b200.so is not built (%s); run `python -m paper_2502_16982_b200.build`" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    L.muon_workspace_bytes.argtypes = [C.POINTER(muon_group), C.c_int, C.POINTER(C.c_size_t)]
    L.muon_partition.argtypes = [C.POINTER(muon_group), C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_double)]
    L.muon_partition_slots.argtypes = [C.POINTER(muon_group), C.c_int, C.c_int, C.POINTER(C.c_int),
                                       C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_double)]
    L.muon_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(muon_group), C.c_int, C.c_void_p, C.c_size_t, C.c_int]
    L.muon_step.argtypes = [C.c_void_p, C.POINTER(muon_hparams), C.c_void_p]
    L.muon_plan_buckets.argtypes = [C.POINTER(muon_group), C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    L.muon_plan_flops.argtypes = [C.POINTER(muon_group), C.c_int, C.c_int, C.POINTER(C.c_double),
                                  C.POINTER(C.c_double)]
    L.muon_plan_work.argtypes = [C.POINTER(muon_group), C.c_int, C.c_int, C.POINTER(C.c_double),
                                 C.POINTER(C.c_double)]
    L.muon_debug_tile_table.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int16), C.c_int,
                                        C.POINTER(C.c_int), C.POINTER(C.c_int)]
    L.muon_step_bucket.argtypes = [C.c_void_p, C.POINTER(muon_hparams), C.c_int, C.c_void_p]
    L.muon_step_host.argtypes = [C.c_void_p, C.POINTER(muon_hparams), C.POINTER(C.POINTER(C.c_void_p)),
                                 C.POINTER(C.POINTER(C.c_void_p)), C.c_void_p]
    L.muon_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    L.muon_get_norms.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_float), C.c_int]
    L.muon_get_update_rms.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_float), C.c_int]
    L.muon_destroy.argtypes = [C.c_void_p]
    L.muon_last_error.restype = C.c_char_p
    L.muon_last_launch_count.argtypes = [C.c_void_p]
    L.muon_debug_keep.argtypes = [C.c_void_p, C.c_int]
    L.muon_debug_read.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t]
    L.muon_debug_tmem_bases.argtypes = [C.c_void_p, C.POINTER(C.c_uint), C.c_int]
    L.muon_profile_enable.argtypes = [C.c_void_p, C.c_int]
    L.muon_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int)]
    L.muon_momentum_norm_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_int64,
                                            C.c_int, C.c_float, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
    L.muon_debug_set_chunk_bytes.argtypes = [C.c_size_t]
    L.muon_debug_set_pair_fold.argtypes = [C.c_int]
    L.muon_debug_set_tile_mode.argtypes = [C.c_int]
    L.muon_debug_wait_expiry.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_uint]
    L.muon_adamw_step.argtypes = [C.POINTER(muon_adamw_tensor), C.c_int, C.POINTER(muon_adamw_hparams), C.c_int,
                                  C.c_void_p]
    for name in EXPORTED:
        if name == "muon_debug_set_chunk_bytes":
            getattr(L, name).restype = C.c_size_t
        elif name != "muon_last_error":
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(rc):
    if rc != 0:
        raise MuonError(rc, lib().muon_last_error().decode())


def muon_last_error() -> str:
    return lib().muon_last_error().decode()


@dataclass
class Hyper:
    """Hyper-parameters of one step; defaults are the paper's."""
    lr: float = 2e-2
    wd: float = 0.1
    mu: float = 0.95
    nesterov: bool = True
    ns_steps: int = 5
    a: float = 3.4445
    b: float = -4.7750
    c: float = 2.0315
    eps: float = 1e-7
    rms_scale: float = 0.2
    scale_mode: int = MUON_SCALE_ADJUSTED_LR
    scale_dim: float = 0.0
    coeffs: Optional[Sequence] = None  # one (a, b, c) per Newton-Schulz step
    protect_momentum: bool = False  # a matrix with a non-finite gradient keeps its momentum too

    def to_c(self) -> muon_hparams:
        hp = muon_hparams(self.lr, self.wd, self.mu, int(bool(self.nesterov)), int(self.ns_steps),
                          self.a, self.b, self.c, self.eps, self.rms_scale, int(self.scale_mode),
                          float(self.scale_dim), None, int(bool(self.protect_momentum)))
        if self.coeffs is not None:
            flat = [float(v) for triple in self.coeffs for v in triple]
            if len(flat) != 3 * int(self.ns_steps):
                raise MuonError(MUON_ERR_INVALID_ARG, "coeffs must hold one (a, b, c) per Newton-Schulz step")
            self._coeffs_c = (C.c_float * len(flat))(*flat)  # kept alive by the Hyper object
            hp.coeffs = C.cast(self._coeffs_c, C.POINTER(C.c_float))
        return hp


def _dtype_code(t):
    import torch
    if t.dtype == torch.bfloat16:
        return MUON_DTYPE_BF16
    if t.dtype == torch.float32:
        return MUON_DTYPE_FP32
    raise MuonError(MUON_ERR_UNSUPPORTED, "dtype %s" % t.dtype)


class _GroupArrays:
    """Keeps the ctypes arrays of one param group alive."""

    def __init__(self, ws, gs, ms, shadows=None):
        w0, g0, m0 = ws[0], gs[0], ms[0]
        n = len(ws)
        if shadows is not None:
            import torch
            for t in shadows:
                if t.shape != w0.shape or t.dtype != torch.bfloat16 or t.stride(1) != 1 or t.stride(0) != shadows[0].stride(0):
                    raise MuonError(MUON_ERR_INVALID_ARG, "shadow copies must be bf16, shaped like W, with one row stride")
        for t in list(ws) + list(gs) + list(ms):
            if t.dim() != 2 or t.shape != w0.shape or t.stride(1) != 1:
                raise MuonError(MUON_ERR_INVALID_ARG, "matrices of a group must be 2-D, equal-shaped, rows contiguous")
        for seq, ref in ((ws, w0), (gs, g0), (ms, m0)):
            for t in seq:
                if t.dtype != ref.dtype or t.stride(0) != ref.stride(0):
                    raise MuonError(MUON_ERR_INVALID_ARG, "dtype and row stride must be uniform within a group")
        self.w = (C.c_void_p * n)(*[t.data_ptr() for t in ws])
        self.g = (C.c_void_p * n)(*[t.data_ptr() for t in gs])
        self.m = (C.c_void_p * n)(*[t.data_ptr() for t in ms])
        self.desc = muon_group(
            w0.shape[0], w0.shape[1], n, _dtype_code(w0), _dtype_code(g0), 0,
            C.cast(self.w, C.POINTER(C.c_void_p)), C.cast(self.g, C.POINTER(C.c_void_p)),
            C.cast(self.m, C.POINTER(C.c_void_p)),
            w0.stride(0) if w0.shape[0] > 1 else max(w0.stride(0), w0.shape[1]),
            g0.stride(0) if g0.shape[0] > 1 else max(g0.stride(0), g0.shape[1]),
            m0.stride(0) if m0.shape[0] > 1 else max(m0.stride(0), m0.shape[1]),
            None, 0)
        if shadows is not None:
            s0 = shadows[0]
            self.s = (C.c_void_p * n)(*[t.data_ptr() for t in shadows])
            self.desc.w_shadow = C.cast(self.s, C.POINTER(C.c_void_p))
            self.desc.ld_shadow = s0.stride(0) if s0.shape[0] > 1 else max(s0.stride(0), s0.shape[1])


def shape_only_groups(shapes) -> "C.Array":
    """muon_group array carrying only (rows, cols, count, w_dtype, g_dtype)
    for muon_workspace_bytes."""
    arr = (muon_group * len(shapes))()
    for i, (rows, cols, count, wd, gd) in enumerate(shapes):
        arr[i].rows, arr[i].cols, arr[i].count, arr[i].w_dtype, arr[i].g_dtype = rows, cols, count, wd, gd
    return arr


def muon_workspace_bytes(groups_c, n_groups) -> int:
    out = C.c_size_t(0)
    _check(lib().muon_workspace_bytes(groups_c, n_groups, C.byref(out)))
    return out.value


def muon_momentum_norm_static(g, m, mu: float, nesterov: bool, norm_out, stream=None):
    """M <- mu*M + G in place and ``norm_out[0] = ||U||_F`` for one 2-D CUDA
    matrix, through the entry point that needs no workspace: the library's
    built-in scratch array is used, so nothing is allocated here either
    (``norm_out`` is a one-element fp32 CUDA tensor the caller already owns).
    Meant for callers that cannot get device memory of their own, e.g. because
    the framework's pool has reserved the whole GPU.  Calls on one GPU share
    the scratch: keep them on one stream."""
    import torch
    if g.dim() != 2 or m.shape != g.shape or g.stride(1) != 1 or m.stride(1) != 1:
        raise MuonError(MUON_ERR_INVALID_ARG, "g and m must be equal-shaped 2-D tensors with contiguous rows")
    if m.dtype != torch.float32 or norm_out.dtype != torch.float32:
        raise MuonError(MUON_ERR_INVALID_ARG, "m and norm_out must be fp32")
    dev = g.device.index
    s = torch.cuda.current_stream(dev) if stream is None else stream
    rows, cols = g.shape
    ld_g = g.stride(0) if rows > 1 else max(g.stride(0), cols)
    ld_m = m.stride(0) if rows > 1 else max(m.stride(0), cols)
    _check(lib().muon_momentum_norm_static(
        C.c_void_p(g.data_ptr()), C.c_void_p(m.data_ptr()), rows, cols, ld_g, ld_m, _dtype_code(g),
        float(mu), int(bool(nesterov)), C.c_void_p(norm_out.data_ptr()), dev, C.c_void_p(s.cuda_stream)))


def muon_adamw_step(params, grads, exp_avgs, exp_avg_sqs, step: int, lr: float, wd: float,
                    beta1: float = 0.9, beta2: float = 0.95, eps: float = 1e-8, stream=None):
    """AdamW step over lists of contiguous CUDA tensors (p bf16/fp32, g bf16/fp32,
    m and v fp32), in place; argument marshalling only."""
    import torch
    n = len(params)
    arr = (muon_adamw_tensor * n)()
    for i, (p, g, m, v) in enumerate(zip(params, grads, exp_avgs, exp_avg_sqs)):
        for t in (p, g, m, v):
            if not t.is_contiguous() or t.numel() != p.numel():
                raise MuonError(MUON_ERR_INVALID_ARG, "AdamW tensors must be contiguous and equally sized")
        if m.dtype != torch.float32 or v.dtype != torch.float32:
            raise MuonError(MUON_ERR_INVALID_ARG, "AdamW moments must be fp32")
        arr[i] = muon_adamw_tensor(p.data_ptr(), g.data_ptr(), m.data_ptr(), v.data_ptr(), p.numel(),
                                   _dtype_code(p), _dtype_code(g))
    dev = params[0].device.index
    s = torch.cuda.current_stream(dev) if stream is None else stream
    hp = muon_adamw_hparams(lr, wd, beta1, beta2, eps, int(step))
    _check(lib().muon_adamw_step(arr, n, C.byref(hp), dev, C.c_void_p(s.cuda_stream)))


def muon_partition(shapes, world: int):
    """Owner rank of every matrix for `world` data-parallel ranks.  ``shapes``
    is a list of (rows, cols, count); returns (owners, loads)."""
    arr = shape_only_groups([(r, c, n, MUON_DTYPE_BF16, MUON_DTYPE_BF16) for (r, c, n) in shapes])
    total = sum(n for (_, _, n) in shapes)
    owners = (C.c_int * total)()
    loads = (C.c_double * world)()
    _check(lib().muon_partition(arr, len(shapes), int(world), owners, loads))
    return list(owners), list(loads)


def muon_partition_slots(shapes, world: int):
    """Slot partition for in-place collectives.  ``shapes`` is a list of (rows,
    cols, count, w_dtype code, g_dtype code); returns (owner per matrix, position
    in the owner's slot per matrix, slot capacity per bucket, load per rank)."""
    arr = shape_only_groups(shapes)
    total = sum(sh[2] for sh in shapes)
    _, n_buckets = muon_plan_buckets(shapes)
    owners = (C.c_int * total)()
    pos = (C.c_int * total)()
    share = (C.c_int * n_buckets)()
    loads = (C.c_double * world)()
    _check(lib().muon_partition_slots(arr, len(shapes), int(world), owners, pos, share, loads))
    return list(owners), list(pos), list(share), list(loads)


def muon_plan_flops(shapes, ns_steps: int = 5):
    """(algorithmic, planned) Newton-Schulz FLOPs of one step; ``shapes`` is a
    list of (rows, cols, count)."""
    arr = shape_only_groups([(r, c, n, MUON_DTYPE_BF16, MUON_DTYPE_BF16) for (r, c, n) in shapes])
    alg, planned = C.c_double(0), C.c_double(0)
    _check(lib().muon_plan_flops(arr, len(shapes), int(ns_steps), C.byref(alg), C.byref(planned)))
    return alg.value, planned.value


def muon_plan_work(shapes, ns_steps: int = 5):
    """({kind: planned FLOPs}, {kind: executed FLOPs}) of one step per kernel
    kind; ``shapes`` is a list of (rows, cols, count).  Executed counts whole
    tiles: padding and dropped blocks included."""
    arr = shape_only_groups([(r, c, n, MUON_DTYPE_BF16, MUON_DTYPE_BF16) for (r, c, n) in shapes])
    planned = (C.c_double * len(KERNEL_KINDS))()
    executed = (C.c_double * len(KERNEL_KINDS))()
    _check(lib().muon_plan_work(arr, len(shapes), int(ns_steps), planned, executed))
    return ({k: planned[i] for i, k in enumerate(KERNEL_KINDS)},
            {k: executed[i] for i, k in enumerate(KERNEL_KINDS)})


def muon_debug_tile_table(rows: int, cols: int, which: int, count: int = 4096):
    """(tiles, matrices per unit) of a bucket of ``count`` matrices (few small
    matrices are cut into finer tiles): every tile is a dict with the row blocks
    ``i`` and matrices ``dm`` of the two CTAs, the column blocks ``j`` of the
    two accumulator halves, the width ``nbw`` and the ``keep`` masks."""
    n, unit = C.c_int(0), C.c_int(0)
    _check(lib().muon_debug_tile_table(rows, cols, count, which, None, 0, C.byref(n), C.byref(unit)))
    buf = (C.c_int16 * (10 * max(1, n.value)))()
    _check(lib().muon_debug_tile_table(rows, cols, count, which, buf, n.value, C.byref(n), C.byref(unit)))
    tiles = []
    for k in range(n.value):
        v = buf[10 * k:10 * k + 10]
        tiles.append({"i": (v[0], v[1]), "j": (v[2], v[3]), "nbw": v[4], "dm": (v[5], v[6]), "keep": (v[7], v[8]),
                      "half": v[9]})
    return tiles, unit.value


def muon_debug_set_tile_mode(mode: int) -> int:
    """How tiles are cut where row blocks do not pair up (bit 0: half-height
    tiles for a row block without a partner, bit 1: for lone diagonal blocks of
    symmetric products; default 1).  Returns the previous mode."""
    return lib().muon_debug_set_tile_mode(int(mode))


def muon_debug_set_pair_fold(mode: int) -> int:
    """Where two iterations are taken per pass over X: 0 = the first two, by
    shape (default), 1 = never, 2 = the first two whenever the short side is at
    least 16, 3 = every pair for wide matrices, 4 = every pair whenever the
    short side is at least 16.  Returns the previous mode."""
    return lib().muon_debug_set_pair_fold(int(mode))


def muon_plan_buckets(shapes):
    """Bucket of every matrix.  ``shapes`` is a list of (rows, cols, count,
    w_dtype code, g_dtype code); returns (bucket per matrix, number of buckets)."""
    arr = shape_only_groups(shapes)
    total = sum(sh[2] for sh in shapes)
    out = (C.c_int * total)()
    n = C.c_int(0)
    _check(lib().muon_plan_buckets(arr, len(shapes), out, C.byref(n)))
    return list(out), n.value


def muon_debug_set_chunk_bytes(nbytes: int) -> int:
    """Test knob: bound on the Newton-Schulz operand bytes of one bucket chunk
    (0 = default).  Returns the previous value."""
    return lib().muon_debug_set_chunk_bytes(int(nbytes))


class MuonContext:
    """One initialised set of param groups.

    ``groups`` is a list of (weights, grads, momenta) triples, or
    (weights, grads, momenta, shadows) with bf16 copies of fp32 weights; each
    entry is a list of equal-shaped 2-D CUDA tensors (bf16 or fp32 weights and
    gradients, fp32 momenta).  Tensors must outlive the context.
    """

    def __init__(self, groups: Sequence[Sequence[Sequence["torch.Tensor"]]], device: Optional[int] = None,
                 workspace: Optional["torch.Tensor"] = None):
        """``workspace``: an optional uint8 CUDA tensor to carve the library's
        workspace from (at least ``muon_workspace_bytes`` + 1023 bytes, so that a
        1024-byte aligned start fits); by default one is allocated here."""
        import torch
        if not torch.cuda.is_available():
            raise MuonError(MUON_ERR_CUDA, "no CUDA device: this library has no CPU path")
        L = lib()
        self._arrays: List[_GroupArrays] = [_GroupArrays(*g) for g in groups]
        self._tensors = groups
        n = len(self._arrays)
        self._groups_c = (muon_group * n)(*[a.desc for a in self._arrays])
        self.n_groups = n
        self.n_matrices = sum(a.desc.count for a in self._arrays)
        dev = groups[0][0][0].device
        self.device = dev.index if device is None else device
        nbytes = muon_workspace_bytes(self._groups_c, n)
        self.workspace_bytes = nbytes
        if workspace is None:
            workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
        elif workspace.dtype != torch.uint8 or not workspace.is_contiguous() or workspace.device != dev:
            raise MuonError(MUON_ERR_WORKSPACE, "workspace must be a contiguous uint8 tensor on the matrices' device")
        self.workspace = workspace
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 1023) // 1024 * 1024
        if self._ws_ptr + nbytes > base + workspace.numel():
            raise MuonError(MUON_ERR_WORKSPACE, "workspace too small: need %d bytes after alignment" % nbytes)
        ctx = C.c_void_p()
        _check(L.muon_init(C.byref(ctx), self._groups_c, n, C.c_void_p(self._ws_ptr), nbytes, self.device))
        self._ctx = ctx

    # -- the C calls -------------------------------------------------------
    def muon_step(self, hp: Hyper, stream=None):
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        c_hp = hp.to_c()
        _check(lib().muon_step(self._ctx, C.byref(c_hp), C.c_void_p(s.cuda_stream)))

    def muon_step_bucket(self, hp: Hyper, bucket: int, stream=None):
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        c_hp = hp.to_c()
        _check(lib().muon_step_bucket(self._ctx, C.byref(c_hp), int(bucket), C.c_void_p(s.cuda_stream)))

    def muon_step_host(self, hp: Hyper, g_host, w_host=None, stream=None):
        """g_host / w_host: per group, a list of pinned CPU tensors (dense)."""
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        c_hp = hp.to_c()

        def table(host):
            rows = [(C.c_void_p * len(ts))(*[t.data_ptr() for t in ts]) for ts in host]
            tab = (C.POINTER(C.c_void_p) * len(rows))(*[C.cast(r, C.POINTER(C.c_void_p)) for r in rows])
            return rows, tab

        g_rows, g_tab = table(g_host)
        w_tab = None
        if w_host is not None:
            w_rows, w_tab = table(w_host)
        _check(lib().muon_step_host(self._ctx, C.byref(c_hp), g_tab, w_tab, C.c_void_p(s.cuda_stream)))

    def muon_status(self, stream=None):
        """Synchronises the stream; returns (status_code, matrix_index)."""
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        st, mi = C.c_int(0), C.c_int(-1)
        _check(lib().muon_status(self._ctx, C.c_void_p(s.cuda_stream), C.byref(st), C.byref(mi)))
        return st.value, mi.value

    def muon_get_norms(self, stream=None):
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        out = (C.c_float * self.n_matrices)()
        _check(lib().muon_get_norms(self._ctx, C.c_void_p(s.cuda_stream), out, self.n_matrices))
        return list(out)

    def muon_get_update_rms(self, stream=None):
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        out = (C.c_float * self.n_matrices)()
        _check(lib().muon_get_update_rms(self._ctx, C.c_void_p(s.cuda_stream), out, self.n_matrices))
        return list(out)

    def muon_last_launch_count(self) -> int:
        return lib().muon_last_launch_count(self._ctx)

    def muon_profile_enable(self, enable: bool):
        _check(lib().muon_profile_enable(self._ctx, int(enable)))

    def muon_profile_read(self):
        """Returns {kernel kind: (milliseconds, launches)} since the last read."""
        n = len(KERNEL_KINDS)
        ms = (C.c_double * n)()
        cnt = (C.c_int * n)()
        _check(lib().muon_profile_read(self._ctx, ms, cnt))
        return {k: (ms[i], cnt[i]) for i, k in enumerate(KERNEL_KINDS)}

    def muon_debug_tmem_bases(self, n: int = 296):
        out = (C.c_uint * n)()
        _check(lib().muon_debug_tmem_bases(self._ctx, out, n))
        return list(out)

    def muon_debug_wait_expiry(self, matrix_index: int, limit_ms: int = 20, stream=None):
        import torch
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().muon_debug_wait_expiry(self._ctx, C.c_void_p(s.cuda_stream), int(matrix_index), int(limit_ms)))

    def muon_debug_keep(self, keep: bool):
        _check(lib().muon_debug_keep(self._ctx, int(keep)))

    def muon_debug_read(self, matrix_index: int, which: int, rows: int, cols: int):
        """Returns a CPU bf16 tensor rows x cols (short side first)."""
        import torch
        out = torch.empty((rows, cols), dtype=torch.bfloat16)
        _check(lib().muon_debug_read(self._ctx, matrix_index, which, C.c_void_p(out.data_ptr()), out.numel() * 2))
        return out

    def muon_destroy(self):
        if getattr(self, "_ctx", None) is not None and self._ctx:
            lib().muon_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.muon_destroy()
        except Exception:
            pass
