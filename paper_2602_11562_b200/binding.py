"""ctypes binding of liblaser.so: same names as the C entry points, torch tensors in place of raw pointers.

Only marshalling happens here (pointer extraction, shape / dtype / contiguity checks, workspace and output
allocation through torch).  Every arithmetic step of the path runs inside the library's CUDA kernels.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_STREAM = 0, 1, 2, 3
DTYPE_F32, DTYPE_BF16 = 0, 1

_LIB: Optional[ctypes.CDLL] = None


class LaserError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {laser_status_string(status)} (status {status})")


class LaserConfig(ctypes.Structure):
    """Mirror of `laser_config` in include/laser.h."""
    _fields_ = [
        ("num_users", ctypes.c_int32), ("max_len", ctypes.c_int32), ("d_model", ctypes.c_int32),
        ("d_qk", ctypes.c_int32), ("num_heads", ctypes.c_int32), ("seg_size", ctypes.c_int32),
        ("num_gsta_layers", ctypes.c_int32), ("dtype", ctypes.c_int32), ("total_cands", ctypes.c_int32),
        ("max_cands_per_user", ctypes.c_int32), ("path", ctypes.c_int32),
        ("sta_gamma", ctypes.c_float), ("gsta_scale", ctypes.c_float),
    ]

    @property
    def n_seg(self) -> int:
        return -(-self.max_len // self.seg_size)

    def torch_dtype(self):
        return torch.float32 if self.dtype == DTYPE_F32 else torch.bfloat16


class LaserFfnParams(ctypes.Structure):
    """Mirror of `laser_ffn_params` in include/laser.h."""
    _fields_ = [
        ("d_hidden", ctypes.c_int32), ("ln_eps", ctypes.c_float),
        ("W1", ctypes.c_void_p), ("b1", ctypes.c_void_p), ("W2", ctypes.c_void_p), ("b2", ctypes.c_void_p),
        ("ln_gain", ctypes.c_void_p), ("ln_shift", ctypes.c_void_p),
    ]


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblaser.so")


def load_library() -> ctypes.CDLL:
    """Load liblaser.so (built by `python -m paper_2602_11562_b200.build`). There is no fallback."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2602_11562_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(path)
    vp, i32p, cfgp, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(LaserConfig), ctypes.c_size_t
    lib.laser_workspace_bytes.restype = sz
    lib.laser_workspace_bytes.argtypes = [cfgp]
    lib.laser_host_workspace_bytes.restype = sz
    lib.laser_host_workspace_bytes.argtypes = [cfgp]
    lib.laser_host_transfer_bytes.restype = ctypes.c_int
    lib.laser_host_transfer_bytes.argtypes = [cfgp, vp, i32p, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.laser_sta_forward.restype = ctypes.c_int
    lib.laser_sta_forward.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, vp, sz, vp]
    lib.laser_gsta_forward.restype = ctypes.c_int
    lib.laser_gsta_forward.argtypes = [cfgp, vp, i32p, i32p, vp, vp, vp, vp, sz, vp]
    lib.laser_forward.restype = ctypes.c_int
    lib.laser_forward.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.laser_forward_packed.restype = ctypes.c_int
    lib.laser_forward_packed.argtypes = [cfgp, vp, i32p, i32p, vp, i32p, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.laser_forward_host.restype = ctypes.c_int
    lib.laser_forward_host.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, vp, vp, sz, vp, ctypes.c_int]
    lib.laser_sta_forward_static.restype = ctypes.c_int
    lib.laser_sta_forward_static.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, vp, vp]
    lib.laser_fusion_forward.restype = ctypes.c_int
    lib.laser_fusion_forward.argtypes = [cfgp, vp, vp, i32p, i32p, ctypes.c_int32, vp, vp, sz, vp]
    lib.laser_sta_softmax_workspace_bytes.restype = sz
    lib.laser_sta_softmax_workspace_bytes.argtypes = [cfgp]
    lib.laser_sta_softmax_forward.restype = ctypes.c_int
    lib.laser_sta_softmax_forward.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, vp, sz, vp]
    lib.laser_backward_workspace_bytes.restype = sz
    lib.laser_backward_workspace_bytes.argtypes = [cfgp]
    lib.laser_backward.restype = ctypes.c_int
    lib.laser_backward.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    ffnp = ctypes.POINTER(LaserFfnParams)
    lib.laser_ffn_workspace_bytes.restype = sz
    lib.laser_ffn_workspace_bytes.argtypes = [cfgp, ctypes.c_int32]
    lib.laser_ffn_forward.restype = ctypes.c_int
    lib.laser_ffn_forward.argtypes = [cfgp, ffnp, vp, i32p, i32p, vp, sz, vp]
    lib.laser_forward_ffn.restype = ctypes.c_int
    lib.laser_forward_ffn.argtypes = [cfgp, vp, i32p, vp, i32p, vp, vp, vp, vp, ffnp, vp, vp, vp, sz, vp]
    lib.laser_check_status.restype = ctypes.c_int
    lib.laser_check_status.argtypes = [vp, vp]
    lib.laser_workspace_regions.restype = ctypes.c_int
    lib.laser_workspace_regions.argtypes = [cfgp, ctypes.c_int, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.laser_selftest_wait_timeout.restype = ctypes.c_int
    lib.laser_selftest_wait_timeout.argtypes = [vp, sz, ctypes.c_int32, vp]
    lib.laser_last_launch_count.restype = ctypes.c_int
    lib.laser_last_launch_count.argtypes = []
    lib.laser_profile_enable.restype = ctypes.c_int
    lib.laser_profile_enable.argtypes = [ctypes.c_int]
    lib.laser_profile_read.restype = ctypes.c_int
    lib.laser_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_char_p)]
    lib.laser_status_string.restype = ctypes.c_char_p
    lib.laser_status_string.argtypes = [ctypes.c_int]
    _LIB = lib
    return lib


def make_config(*, num_users, max_len, d_model, d_qk, num_heads, seg_size, num_gsta_layers, dtype, total_cands,
                max_cands_per_user, path=PATH_AUTO, sta_gamma=0.0, gsta_scale=0.0) -> LaserConfig:
    if isinstance(dtype, str):
        dtype = {"f32": DTYPE_F32, "bf16": DTYPE_BF16}[dtype]
    return LaserConfig(num_users, max_len, d_model, d_qk, num_heads, seg_size, num_gsta_layers, dtype, total_cands,
                       max_cands_per_user, path, float(sta_gamma), float(gsta_scale))


def laser_status_string(status: int) -> str:
    return load_library().laser_status_string(int(status)).decode()


def laser_workspace_bytes(cfg: LaserConfig) -> int:
    return int(load_library().laser_workspace_bytes(ctypes.byref(cfg)))


def laser_workspace_regions(cfg: LaserConfig) -> list:
    """[(byte offset, bytes in use)] of the regions a call with this configuration may write inside its workspace."""
    lib = load_library()
    n = lib.laser_workspace_regions(ctypes.byref(cfg), 0, None, None)
    _check(min(n, 0), "laser_workspace_regions")
    offs, sizes = (ctypes.c_size_t * n)(), (ctypes.c_size_t * n)()
    _check(min(lib.laser_workspace_regions(ctypes.byref(cfg), n, offs, sizes), 0), "laser_workspace_regions")
    return [(int(offs[i]), int(sizes[i])) for i in range(n)]


def laser_selftest_wait_timeout(workspace: torch.Tensor, poll_limit: int = 1024, stream=None) -> None:
    """Enqueues the bounded-wait self-test block; laser_check_status(workspace) then returns LASER_ERR_TIMEOUT (-5)."""
    if not workspace.is_cuda or workspace.dtype != torch.uint8:
        raise LaserError(-1, "laser_selftest_wait_timeout (workspace must be a uint8 device tensor)")
    _check(load_library().laser_selftest_wait_timeout(ctypes.c_void_p(workspace.data_ptr()), workspace.numel(),
                                                      int(poll_limit), ctypes.c_void_p(_stream_ptr(stream))),
           "laser_selftest_wait_timeout")


def laser_host_workspace_bytes(cfg: LaserConfig) -> int:
    return int(load_library().laser_host_workspace_bytes(ctypes.byref(cfg)))


def laser_host_transfer_bytes(cfg: LaserConfig, lengths_h, items_h=None) -> tuple:
    """(host-to-device bytes, device-to-host bytes) that laser_forward_host moves for these HOST lengths and this HOST
    items tensor (None: as for pageable memory)."""
    if lengths_h.is_cuda or lengths_h.dtype != torch.int32 or not lengths_h.is_contiguous():
        raise LaserError(-1, "laser_host_transfer_bytes (lengths must be a contiguous int32 HOST tensor)")
    if items_h is not None and items_h.is_cuda:
        raise LaserError(-1, "laser_host_transfer_bytes (items must be a HOST tensor)")
    h2d, d2h = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load_library().laser_host_transfer_bytes(ctypes.byref(cfg),
                                                    ctypes.c_void_p(items_h.data_ptr() if items_h is not None else 0),
                                                    ctypes.c_void_p(lengths_h.data_ptr()), ctypes.byref(h2d),
                                                    ctypes.byref(d2h)), "laser_host_transfer_bytes")
    return int(h2d.value), int(d2h.value)


def laser_last_launch_count() -> int:
    return int(load_library().laser_last_launch_count())


def laser_profile_enable(on: bool) -> None:
    load_library().laser_profile_enable(1 if on else 0)


def laser_profile_read(max_kernels: int = 256):
    """[(kernel name, milliseconds)] of the last profiled call on this thread, in launch order."""
    ms = (ctypes.c_float * max_kernels)()
    names = (ctypes.c_char_p * max_kernels)()
    n = load_library().laser_profile_read(max_kernels, ms, names)
    _check(min(n, 0), "laser_profile_read")
    return [(names[i].decode(), float(ms[i])) for i in range(n)]


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _workspace(cfg: LaserConfig, workspace, device, host: bool = False) -> torch.Tensor:
    need = laser_host_workspace_bytes(cfg) if host else laser_workspace_bytes(cfg)
    if need == 0:
        raise LaserError(-1, "laser_workspace_bytes (invalid or unsupported configuration)")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace


def _check(rc: int, where: str):
    if rc != 0:
        raise LaserError(rc, where)


def laser_sta_forward(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime=None, workspace=None, stream=None):
    """STA: returns H' [N, L', d]. All tensors live on the GPU; see include/laser.h for shapes."""
    lib, dt = load_library(), cfg.torch_dtype()
    ws = _workspace(cfg, workspace, items.device)
    if Hprime is None:
        Hprime = torch.empty((cfg.total_cands, cfg.n_seg, cfg.d_model), dtype=dt, device=items.device)
    rc = lib.laser_sta_forward(ctypes.byref(cfg), _dev(items, dt, "items"), _dev(lengths, torch.int32, "lengths"),
                               _dev(cands, dt, "cands"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                               _dev(Wq, dt, "Wq"), _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"), _dev(Hprime, dt, "Hprime"),
                               ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_sta_forward")
    return Hprime


def laser_sta_forward_static(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, status_out=None,
                             stream=None):
    """STA through the entry point that needs no workspace: for callers that cannot allocate device memory (all
    scratch lives in a fixed array inside the library).  The caller supplies every buffer, including the output
    Hprime [N, L', d] and, optionally, a one-element int32 device tensor that receives the device-side status."""
    lib, dt = load_library(), cfg.torch_dtype()
    rc = lib.laser_sta_forward_static(ctypes.byref(cfg), _dev(items, dt, "items"),
                                      _dev(lengths, torch.int32, "lengths"), _dev(cands, dt, "cands"),
                                      _dev(cand_offsets, torch.int32, "cand_offsets"), _dev(Wq, dt, "Wq"),
                                      _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"), _dev(Hprime, dt, "Hprime"),
                                      None if status_out is None else _dev(status_out, torch.int32, "status_out"),
                                      _stream_ptr(stream))
    _check(rc, "laser_sta_forward_static")
    return Hprime


def laser_gsta_forward(cfg, Hprime, lengths, cand_offsets, cands, Wgsta, z=None, workspace=None, stream=None):
    """GSTA over a given H': returns z [N, d]."""
    lib, dt = load_library(), cfg.torch_dtype()
    ws = _workspace(cfg, workspace, Hprime.device)
    if z is None:
        z = torch.empty((cfg.total_cands, cfg.d_model), dtype=dt, device=Hprime.device)
    rc = lib.laser_gsta_forward(ctypes.byref(cfg), _dev(Hprime, dt, "Hprime"), _dev(lengths, torch.int32, "lengths"),
                                _dev(cand_offsets, torch.int32, "cand_offsets"), _dev(cands, dt, "cands"),
                                _dev(Wgsta, dt, "Wgsta"), _dev(z, dt, "z"), ws.data_ptr(), ws.numel(),
                                _stream_ptr(stream))
    _check(rc, "laser_gsta_forward")
    return z


def laser_forward(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, Hprime=None, z=None, workspace=None,
                  stream=None, want_hprime=False):
    """STA + GSTA: returns z, or (H', z) when want_hprime / an Hprime buffer is given."""
    lib, dt = load_library(), cfg.torch_dtype()
    ws = _workspace(cfg, workspace, items.device)
    if z is None:
        z = torch.empty((cfg.total_cands, cfg.d_model), dtype=dt, device=items.device)
    if Hprime is None and want_hprime:
        Hprime = torch.empty((cfg.total_cands, cfg.n_seg, cfg.d_model), dtype=dt, device=items.device)
    rc = lib.laser_forward(ctypes.byref(cfg), _dev(items, dt, "items"), _dev(lengths, torch.int32, "lengths"),
                           _dev(cands, dt, "cands"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                           _dev(Wq, dt, "Wq"), _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"), _dev(Wgsta, dt, "Wgsta"),
                           None if Hprime is None else _dev(Hprime, dt, "Hprime"), _dev(z, dt, "z"),
                           ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_forward")
    return (Hprime, z) if Hprime is not None else z


def laser_forward_packed(cfg, items_packed, item_offsets, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, Hprime=None,
                         z=None, workspace=None, stream=None, want_hprime=False):
    """laser_forward on items stored without padding: items_packed [item_offsets[U], d], item_offsets [U + 1] int32."""
    lib, dt = load_library(), cfg.torch_dtype()
    ws = _workspace(cfg, workspace, items_packed.device)
    if z is None:
        z = torch.empty((cfg.total_cands, cfg.d_model), dtype=dt, device=items_packed.device)
    if Hprime is None and want_hprime:
        Hprime = torch.empty((cfg.total_cands, cfg.n_seg, cfg.d_model), dtype=dt, device=items_packed.device)
    rc = lib.laser_forward_packed(ctypes.byref(cfg), _dev(items_packed, dt, "items_packed"),
                                  _dev(item_offsets, torch.int32, "item_offsets"), _dev(lengths, torch.int32, "lengths"),
                                  _dev(cands, dt, "cands"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                                  _dev(Wq, dt, "Wq"), _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"), _dev(Wgsta, dt, "Wgsta"),
                                  None if Hprime is None else _dev(Hprime, dt, "Hprime"), _dev(z, dt, "z"),
                                  ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_forward_packed")
    return (Hprime, z) if Hprime is not None else z


def laser_fusion_forward(cfg, Hprime, z, lengths, cand_offsets, num_recent, fused=None, workspace=None, stream=None):
    """Multi-resolution fusion: returns fused [N, (2 + num_recent) * d] = [z | max-pooled H' | most recent segments]."""
    lib, dt = load_library(), cfg.torch_dtype()
    if workspace is None:
        workspace = torch.empty(256, dtype=torch.uint8, device=Hprime.device)
    if fused is None:
        fused = torch.empty((cfg.total_cands, (2 + num_recent) * cfg.d_model), dtype=dt, device=Hprime.device)
    rc = lib.laser_fusion_forward(ctypes.byref(cfg), _dev(Hprime, dt, "Hprime"), _dev(z, dt, "z"),
                                  _dev(lengths, torch.int32, "lengths"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                                  int(num_recent), _dev(fused, dt, "fused"), workspace.data_ptr(), workspace.numel(),
                                  _stream_ptr(stream))
    _check(rc, "laser_fusion_forward")
    return fused


def laser_sta_softmax_workspace_bytes(cfg: LaserConfig) -> int:
    return int(load_library().laser_sta_softmax_workspace_bytes(ctypes.byref(cfg)))


def laser_sta_softmax_forward(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime=None, workspace=None,
                              stream=None):
    """The softmax-aggregation variant of STA (the paper's ablation): returns H' [N, L', d]."""
    lib, dt = load_library(), cfg.torch_dtype()
    need = laser_sta_softmax_workspace_bytes(cfg)
    if need == 0:
        raise LaserError(-1, "laser_sta_softmax_workspace_bytes (invalid or unsupported configuration)")
    ws = torch.empty(need, dtype=torch.uint8, device=items.device) if workspace is None else workspace
    if Hprime is None:
        Hprime = torch.empty((cfg.total_cands, cfg.n_seg, cfg.d_model), dtype=dt, device=items.device)
    rc = lib.laser_sta_softmax_forward(ctypes.byref(cfg), _dev(items, dt, "items"), _dev(lengths, torch.int32, "lengths"),
                                       _dev(cands, dt, "cands"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                                       _dev(Wq, dt, "Wq"), _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"),
                                       _dev(Hprime, dt, "Hprime"), ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_sta_softmax_forward")
    return Hprime


def laser_backward_workspace_bytes(cfg: LaserConfig) -> int:
    return int(load_library().laser_backward_workspace_bytes(ctypes.byref(cfg)))


def laser_backward(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wg, dz, workspace=None, stream=None):
    """Backward pass of laser_forward for the upstream gradient dz [N, d] (float32).  Returns a dict of float32
    tensors: d_items [U, L, d], d_cands [N, d], dWq, dWk [d, d_qk], dWv [d, d], dWg [M, 3, d, d]."""
    lib, dt = load_library(), cfg.torch_dtype()
    need = laser_backward_workspace_bytes(cfg)
    if need == 0:
        raise LaserError(-1, "laser_backward_workspace_bytes (invalid or unsupported configuration)")
    dev = items.device
    ws = torch.empty(need, dtype=torch.uint8, device=dev) if workspace is None else workspace
    f32 = torch.float32
    out = {"d_items": torch.empty((cfg.num_users, cfg.max_len, cfg.d_model), dtype=f32, device=dev),
           "d_cands": torch.empty((cfg.total_cands, cfg.d_model), dtype=f32, device=dev),
           "dWq": torch.empty((cfg.d_model, cfg.d_qk), dtype=f32, device=dev),
           "dWk": torch.empty((cfg.d_model, cfg.d_qk), dtype=f32, device=dev),
           "dWv": torch.empty((cfg.d_model, cfg.d_model), dtype=f32, device=dev),
           "dWg": torch.empty((cfg.num_gsta_layers, 3, cfg.d_model, cfg.d_model), dtype=f32, device=dev)}
    rc = lib.laser_backward(ctypes.byref(cfg), _dev(items, dt, "items"), _dev(lengths, torch.int32, "lengths"),
                            _dev(cands, dt, "cands"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                            _dev(Wq, dt, "Wq"), _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"), _dev(Wg, dt, "Wg"),
                            _dev(dz, f32, "dz"), out["d_items"].data_ptr(), out["d_cands"].data_ptr(),
                            out["dWq"].data_ptr(), out["dWk"].data_ptr(), out["dWv"].data_ptr(), out["dWg"].data_ptr(),
                            ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_backward")
    return out


def laser_ffn_workspace_bytes(cfg: LaserConfig, d_hidden: int) -> int:
    return int(load_library().laser_ffn_workspace_bytes(ctypes.byref(cfg), int(d_hidden)))


def _ffn_params(cfg, ffn: dict, ln_eps: float):
    """ffn: {"W1" [d, hid], "b1" [hid], "W2" [hid, d], "b2" [d], "ln_g" [d], "ln_b" [d]} device tensors."""
    dt = cfg.torch_dtype()
    hid = int(ffn["W1"].shape[1])
    return LaserFfnParams(hid, float(ln_eps), _dev(ffn["W1"], dt, "W1"), _dev(ffn["b1"], dt, "b1"),
                          _dev(ffn["W2"], dt, "W2"), _dev(ffn["b2"], dt, "b2"), _dev(ffn["ln_g"], dt, "ln_g"),
                          _dev(ffn["ln_b"], dt, "ln_b")), hid


def _ffn_workspace(cfg, hid, workspace, device):
    need = laser_ffn_workspace_bytes(cfg, hid)
    if need == 0:
        raise LaserError(-1, "laser_ffn_workspace_bytes (invalid or unsupported configuration)")
    return torch.empty(need, dtype=torch.uint8, device=device) if workspace is None else workspace


def laser_ffn_forward(cfg, ffn, Hprime, lengths, cand_offsets, ln_eps=0.0, workspace=None, stream=None):
    """Eq. 6 in place on H' [N, L', d]: rows of non-empty segments become LN(FFN(s) + s).  Returns Hprime."""
    lib, dt = load_library(), cfg.torch_dtype()
    params, hid = _ffn_params(cfg, ffn, ln_eps)
    ws = _ffn_workspace(cfg, hid, workspace, Hprime.device)
    rc = lib.laser_ffn_forward(ctypes.byref(cfg), ctypes.byref(params), _dev(Hprime, dt, "Hprime"),
                               _dev(lengths, torch.int32, "lengths"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                               ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_ffn_forward")
    return Hprime


def laser_forward_ffn(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, ffn, Hprime=None, z=None,
                      ln_eps=0.0, workspace=None, stream=None, want_hprime=False):
    """STA, Eq. 6 on every segment vector, GSTA: returns z, or (refined H', z)."""
    lib, dt = load_library(), cfg.torch_dtype()
    params, hid = _ffn_params(cfg, ffn, ln_eps)
    ws = _ffn_workspace(cfg, hid, workspace, items.device)
    if z is None:
        z = torch.empty((cfg.total_cands, cfg.d_model), dtype=dt, device=items.device)
    if Hprime is None and want_hprime:
        Hprime = torch.empty((cfg.total_cands, cfg.n_seg, cfg.d_model), dtype=dt, device=items.device)
    rc = lib.laser_forward_ffn(ctypes.byref(cfg), _dev(items, dt, "items"), _dev(lengths, torch.int32, "lengths"),
                               _dev(cands, dt, "cands"), _dev(cand_offsets, torch.int32, "cand_offsets"),
                               _dev(Wq, dt, "Wq"), _dev(Wk, dt, "Wk"), _dev(Wv, dt, "Wv"), _dev(Wgsta, dt, "Wgsta"),
                               ctypes.byref(params), None if Hprime is None else _dev(Hprime, dt, "Hprime"),
                               _dev(z, dt, "z"), ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "laser_forward_ffn")
    return (Hprime, z) if Hprime is not None else z


def _host(t: torch.Tensor, dtype, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{name}: expected a contiguous CPU tensor of {dtype}")
    return t.data_ptr()


def laser_forward_host(cfg, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, z, workspace, stream=None,
                       blocking=True):
    """End-to-end call on HOST tensors (ideally pinned): H2D copies, forward, D2H copy of z, inside the library."""
    lib, dt = load_library(), cfg.torch_dtype()
    rc = lib.laser_forward_host(ctypes.byref(cfg), _host(items, dt, "items"), _host(lengths, torch.int32, "lengths"),
                                _host(cands, dt, "cands"), _host(cand_offsets, torch.int32, "cand_offsets"),
                                _host(Wq, dt, "Wq"), _host(Wk, dt, "Wk"), _host(Wv, dt, "Wv"),
                                _host(Wgsta, dt, "Wgsta"), _host(z, dt, "z"), workspace.data_ptr(), workspace.numel(),
                                _stream_ptr(stream), 1 if blocking else 0)
    _check(rc, "laser_forward_host")
    return z


def laser_check_status(workspace: torch.Tensor, stream=None) -> int:
    """Synchronises the stream and returns the device-side status word (0 = ok)."""
    return int(load_library().laser_check_status(workspace.data_ptr(), _stream_ptr(stream)))


@dataclass
class DeviceBatch:
    """A workload's arrays as device tensors of the configuration dtype, plus the matching laser_config."""
    cfg: LaserConfig
    items: torch.Tensor
    lengths: torch.Tensor
    cands: torch.Tensor
    cand_offsets: torch.Tensor
    Wq: torch.Tensor
    Wk: torch.Tensor
    Wv: torch.Tensor
    Wg: torch.Tensor

    @staticmethod
    def from_numpy(*, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wg, S, H, M, dtype, gamma=0.0, tau=0.0,
                   path=PATH_AUTO, device="cuda", pin_host=False) -> "DeviceBatch":
        import numpy as np
        dt = torch.float32 if dtype in ("f32", DTYPE_F32) else torch.bfloat16
        U, L, d = items.shape
        offs = np.asarray(cand_offsets, dtype=np.int64)
        N = int(offs[-1])
        maxc = int(np.max(offs[1:] - offs[:-1])) if U > 0 else 0
        cfg = make_config(num_users=U, max_len=L, d_model=d, d_qk=Wq.shape[1], num_heads=H, seg_size=S,
                          num_gsta_layers=M, dtype=DTYPE_F32 if dt == torch.float32 else DTYPE_BF16, total_cands=N,
                          max_cands_per_user=maxc, path=path, sta_gamma=gamma, gsta_scale=tau)

        def up(a, tdt):
            t = torch.from_numpy(np.ascontiguousarray(a)).to(tdt)
            if device == "cpu":
                return t.pin_memory() if pin_host else t
            return t.to(device)

        return DeviceBatch(cfg, up(items, dt), up(np.asarray(lengths, dtype=np.int32), torch.int32), up(cands, dt),
                           up(np.asarray(cand_offsets, dtype=np.int32), torch.int32), up(Wq, dt), up(Wk, dt),
                           up(Wv, dt), up(Wg, dt))

    @staticmethod
    def from_workload(w, path=PATH_AUTO, device="cuda", pin_host=False) -> "DeviceBatch":
        s = w.spec
        return DeviceBatch.from_numpy(items=w.items, lengths=w.lengths, cands=w.cands, cand_offsets=w.cand_offsets,
                                      Wq=w.Wq, Wk=w.Wk, Wv=w.Wv, Wg=w.Wg, S=s.S, H=s.H, M=s.M, dtype=s.dtype,
                                      gamma=w.gamma, tau=w.tau, path=path, device=device, pin_host=pin_host)

    def args(self):
        return (self.items, self.lengths, self.cands, self.cand_offsets, self.Wq, self.Wk, self.Wv)
