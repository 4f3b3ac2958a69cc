"""ctypes binding of the LESS C-ABI library (include/less.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  The functions carry the C names.  There is no CPU fallback: loading
fails loudly when the library has not been built, and nothing here computes.
torch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

from . import build as _build

LESS_OK = 0
LESS_SCORE_NORM_SPARSE = 1
LESS_NO_STATE = 2
LESS_POLICY_LAMBDA = 4
LESS_POLICY_TOVA = 8
LESS_WITH_PARALLEL_FORM = 16
LESS_OUT_F16 = 32

EXPORTED = [
    "less_arena_bytes", "less_create", "less_prefill", "less_decode_step", "less_position",
    "less_state_record_bytes", "less_export_state", "less_import_state",
    "less_read_feature_maps", "less_poll_status", "less_launch_count", "less_strerror",
    "less_destroy", "less_decode_step_host", "less_profile", "less_profile_read",
    "less_prompt_scores_noalloc", "less_masked_attention", "less_kernel_variant",
    "less_last_status_where", "less_selftest_wait_timeout",
]
LESS_NOALLOC_MAX_ROWS = 65536
LESS_ERR_NOALLOC_TOO_LARGE = -12

KERNEL_NAMES = ["feature_map", "decode", "rowstat", "colsum", "attn_out", "select", "build", "finalize",
                "psi", "gather", "masked_pack", "masked_out"]


class less_config(C.Structure):
    _fields_ = [("batch", C.c_int32), ("layers", C.c_int32), ("heads", C.c_int32),
                ("head_dim", C.c_int32), ("rank", C.c_int32), ("hidden", C.c_int32),
                ("heavy", C.c_int32), ("recent", C.c_int32), ("max_prompt", C.c_int32),
                ("max_prefill_layers", C.c_int32), ("flags", C.c_uint32), ("group", C.c_int32)]


class less_weights(C.Structure):
    _fields_ = [("w_phi1", C.c_void_p), ("w_phi2", C.c_void_p), ("w_psi1", C.c_void_p),
                ("w_psi2", C.c_void_p), ("w_psi3", C.c_void_p), ("psi_scale", C.c_void_p)]


class LessError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {less_strerror(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """Loads libless_b200.so (built in-tree).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} is missing: build it with `python -m paper_2402_09398_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(path)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    L.less_arena_bytes.restype = sz
    L.less_arena_bytes.argtypes = [C.POINTER(less_config)]
    L.less_state_record_bytes.restype = sz
    L.less_state_record_bytes.argtypes = [C.POINTER(less_config)]
    L.less_create.restype = C.c_int
    L.less_create.argtypes = [C.POINTER(less_config), C.POINTER(less_weights), vp, sz, C.POINTER(vp)]
    L.less_prefill.restype = C.c_int
    L.less_prefill.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    L.less_decode_step.restype = C.c_int
    L.less_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.less_decode_step_host.restype = C.c_int
    L.less_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp]
    L.less_profile.restype = C.c_int
    L.less_profile.argtypes = [vp, C.c_int]
    L.less_profile_read.restype = C.c_int
    L.less_profile_read.argtypes = [vp, vp, vp]
    L.less_prompt_scores_noalloc.restype = C.c_int
    L.less_prompt_scores_noalloc.argtypes = [vp, vp, i32, i32, vp, vp]
    L.less_position.restype = i64
    L.less_position.argtypes = [vp]
    L.less_launch_count.restype = i64
    L.less_launch_count.argtypes = [vp]
    L.less_export_state.restype = C.c_int
    L.less_export_state.argtypes = [vp, vp, i32, vp, sz, vp]
    L.less_import_state.restype = C.c_int
    L.less_import_state.argtypes = [vp, vp, i32, vp, sz, vp]
    L.less_masked_attention.restype = C.c_int
    L.less_masked_attention.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    L.less_read_feature_maps.restype = C.c_int
    L.less_read_feature_maps.argtypes = [vp, vp, vp, vp]
    L.less_poll_status.restype = C.c_int
    L.less_poll_status.argtypes = [vp, vp]
    L.less_strerror.restype = C.c_char_p
    L.less_strerror.argtypes = [C.c_int]
    L.less_destroy.restype = C.c_int
    L.less_destroy.argtypes = [vp]
    L.less_kernel_variant.restype = C.c_char_p
    L.less_kernel_variant.argtypes = [vp, C.c_int]
    L.less_last_status_where.restype = C.c_int
    L.less_last_status_where.argtypes = [vp]
    L.less_selftest_wait_timeout.restype = C.c_int
    L.less_selftest_wait_timeout.argtypes = [vp, C.c_uint32, vp]
    _lib = L
    return L


# --------------------------------------------------------------------------- #
# the C calls, same names
# --------------------------------------------------------------------------- #
def less_strerror(code: int) -> str:
    return lib().less_strerror(int(code)).decode()


def less_arena_bytes(cfg: less_config) -> int:
    return int(lib().less_arena_bytes(C.byref(cfg)))


def less_state_record_bytes(cfg: less_config) -> int:
    return int(lib().less_state_record_bytes(C.byref(cfg)))


def less_create(cfg: less_config, weights: less_weights, arena_ptr: int, arena_bytes: int):
    out = C.c_void_p()
    rc = lib().less_create(C.byref(cfg), C.byref(weights), arena_ptr, arena_bytes, C.byref(out))
    return rc, out


def less_prefill(ctx, layer_begin, layer_count, prompt_len, Q, K, V, attn_out, stream) -> int:
    return lib().less_prefill(ctx, layer_begin, layer_count, prompt_len, Q, K, V, attn_out, stream)


def less_decode_step(ctx, q, k, v, out, evicted_pos, stream) -> int:
    return lib().less_decode_step(ctx, q, k, v, out, evicted_pos, stream)


def less_decode_step_host(ctx, q_host, k_host, v_host, out_host, stream) -> int:
    return lib().less_decode_step_host(ctx, q_host, k_host, v_host, out_host, stream)


def less_profile(ctx, enable: int) -> int:
    return lib().less_profile(ctx, int(enable))


def less_profile_read(ctx, ms_ptr, launches_ptr) -> int:
    return lib().less_profile_read(ctx, ms_ptr, launches_ptr)


def less_prompt_scores_noalloc(Q, K, n_inst, prompt_len, acc_out, stream) -> int:
    """H2O prompt scores for callers that cannot allocate device memory (a
    process whose pool owns the GPU, a plugin handed only buffers and a stream):
    the scratch lives in a fixed array inside the library.  Device pointers in,
    return code out; at most LESS_NOALLOC_MAX_ROWS rows (n_inst * prompt_len);
    calls that may overlap on the GPU race on the shared array."""
    return lib().less_prompt_scores_noalloc(Q, K, n_inst, prompt_len, acc_out, stream)


def less_position(ctx) -> int:
    return int(lib().less_position(ctx))


def less_launch_count(ctx) -> int:
    return int(lib().less_launch_count(ctx))


def less_export_state(ctx, inst_ptr, n, host_ptr, nbytes, stream) -> int:
    return lib().less_export_state(ctx, inst_ptr, n, host_ptr, nbytes, stream)


def less_import_state(ctx, inst_ptr, n, host_ptr, nbytes, stream) -> int:
    return lib().less_import_state(ctx, inst_ptr, n, host_ptr, nbytes, stream)


def less_masked_attention(ctx, layer_begin, layer_count, seq_len, Q, K, V, exact_until, out, stream) -> int:
    return lib().less_masked_attention(ctx, layer_begin, layer_count, seq_len, Q, K, V, exact_until, out, stream)


def less_read_feature_maps(ctx, phi_ptr, psi_ptr, stream) -> int:
    return lib().less_read_feature_maps(ctx, phi_ptr, psi_ptr, stream)


def less_poll_status(ctx, stream) -> int:
    return lib().less_poll_status(ctx, stream)


def less_destroy(ctx) -> int:
    return lib().less_destroy(ctx)


def less_kernel_variant(ctx, kernel_id: int) -> str:
    return lib().less_kernel_variant(ctx, int(kernel_id)).decode()


def less_last_status_where(ctx) -> int:
    return int(lib().less_last_status_where(ctx))


def less_selftest_wait_timeout(ctx, polls: int, stream) -> int:
    return lib().less_selftest_wait_timeout(ctx, int(polls), stream)


# --------------------------------------------------------------------------- #
# convenience holder: owns the torch buffers the context borrows
# --------------------------------------------------------------------------- #
def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check(rc: int, where: str) -> None:
    if rc != LESS_OK:
        raise LessError(rc, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class LessContext:
    """Allocates the arena with torch, keeps the weights alive, forwards calls."""

    def __init__(self, batch, layers, heads, head_dim, rank, hidden, heavy, recent, max_prompt,
                 weights: Dict[str, torch.Tensor], max_prefill_layers: int = 1, flags: int = 0,
                 psi_scale: Optional[torch.Tensor] = None, device="cuda", group: int = 1):
        if not torch.cuda.is_available():
            raise RuntimeError("the LESS library needs a CUDA device (there is no CPU path)")
        lib()
        self.device = torch.device(device)
        self.cfg = less_config(batch, layers, heads, head_dim, rank, hidden, heavy, recent,
                               max_prompt, max_prefill_layers, flags, group)
        nbytes = less_arena_bytes(self.cfg)
        if nbytes == 0:
            raise LessError(-1, "less_arena_bytes")
        self.weights = {k: v.to(self.device).contiguous() for k, v in weights.items()}
        self.psi_scale = None if psi_scale is None else psi_scale.to(self.device, torch.float32).contiguous()
        self.arena = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        w = less_weights(*(self.weights[n].data_ptr() for n in
                           ("w_phi1", "w_phi2", "w_psi1", "w_psi2", "w_psi3")), _ptr(self.psi_scale))
        torch.cuda.synchronize()
        rc, ctx = less_create(self.cfg, w, self.arena.data_ptr(), nbytes)
        _check(rc, "less_create")
        self.ctx = ctx
        self.instances = batch * layers * heads
        self.group = max(1, group)
        self.N = heavy + recent
        self.record_bytes = less_state_record_bytes(self.cfg)
        self.out_dtype = torch.float16 if flags & LESS_OUT_F16 else torch.float32

    # -- hot path ---------------------------------------------------------- #
    def prefill(self, Q, K, V, layer_begin=0, attn_out=None, stream=None):
        B, Lc, H, S, D = Q.shape
        assert Q.dtype == K.dtype == V.dtype == torch.float16
        assert Q.is_contiguous() and K.is_contiguous() and V.is_contiguous()
        _check(less_prefill(self.ctx, layer_begin, Lc, S, _ptr(Q), _ptr(K), _ptr(V), _ptr(attn_out),
                            _stream_ptr(stream)), "less_prefill")

    def masked_attention(self, Q, K, V, exact_until, layer_begin=0, out=None, stream=None):
        """The parallel form: Q fp16 [B, Lc, H * group, S, D], K, V fp16 [B, Lc, H, S, D], exact_until int32
        [B, Lc, H, S]; the result has Q's shape."""
        B, Lc, _, S, D = Q.shape
        assert Q.dtype == K.dtype == V.dtype == torch.float16 and exact_until.dtype == torch.int32
        assert Q.is_contiguous() and K.is_contiguous() and V.is_contiguous() and exact_until.is_contiguous()
        if out is None:
            out = torch.empty(Q.shape, dtype=torch.float32, device=Q.device)
        _check(less_masked_attention(self.ctx, layer_begin, Lc, S, _ptr(Q), _ptr(K), _ptr(V), _ptr(exact_until),
                                     _ptr(out), _stream_ptr(stream)), "less_masked_attention")
        return out

    def reset(self, layer_begin=0, layer_count=None, stream=None):
        n = self.cfg.layers - layer_begin if layer_count is None else layer_count
        _check(less_prefill(self.ctx, layer_begin, n, 0, None, None, None, None, _stream_ptr(stream)),
               "less_prefill(reset)")

    def decode_step(self, q, k, v, out=None, evicted_pos=None, stream=None):
        assert q.dtype == k.dtype == v.dtype == torch.float16
        if out is None:
            out = torch.empty(q.shape, dtype=self.out_dtype, device=q.device)
        assert out.dtype == self.out_dtype
        _check(less_decode_step(self.ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(evicted_pos),
                                _stream_ptr(stream)), "less_decode_step")
        return out

    def decode_step_host(self, q, k, v, out, stream=None):
        """q, k, v, out: host tensors (pinned for speed); synchronous."""
        _check(less_decode_step_host(self.ctx, _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                     _stream_ptr(stream)), "less_decode_step_host")
        return out

    def profile(self, enable: bool):
        _check(less_profile(self.ctx, 1 if enable else 0), "less_profile")

    def profile_read(self):
        ms = np.zeros(len(KERNEL_NAMES), dtype=np.float32)
        n = np.zeros(len(KERNEL_NAMES), dtype=np.int64)
        _check(less_profile_read(self.ctx, ms.ctypes.data, n.ctypes.data), "less_profile_read")
        return {k: (float(a), int(b)) for k, a, b in zip(KERNEL_NAMES, ms, n)}

    # -- state ------------------------------------------------------------- #
    @property
    def position(self) -> int:
        return less_position(self.ctx)

    @property
    def launches(self) -> int:
        return less_launch_count(self.ctx)

    def _record_views(self, buf: np.ndarray, i: int):
        N, D, R = self.N, self.cfg.head_dim, self.cfg.rank
        rec = buf[i * self.record_bytes:(i + 1) * self.record_bytes]
        off = 16
        views = {"header": rec[:16].view(np.int32)}
        for name, dt, shape in (("pos", np.int32, (N,)), ("acc", np.float32, (N,)),
                                ("K", np.float16, (N, D)), ("V", np.float16, (N, D)),
                                ("psi", np.float32, (N, R)), ("H", np.float32, (R, D)),
                                ("z", np.float32, (R,))):
            n = int(np.prod(shape)) * np.dtype(dt).itemsize
            views[name] = rec[off:off + n].view(dt).reshape(shape)
            off += n
        return views

    def export_state(self, instances: Sequence[int], stream=None):
        inst = np.ascontiguousarray(instances, dtype=np.int32)
        buf = np.zeros(len(inst) * self.record_bytes, dtype=np.uint8)
        _check(less_export_state(self.ctx, inst.ctypes.data, len(inst), buf.ctypes.data, buf.nbytes,
                                 _stream_ptr(stream)), "less_export_state")
        out = []
        for i in range(len(inst)):
            v = self._record_views(buf, i)
            cnt = int(v["header"][0])
            out.append({"count": cnt, "t": int(v["header"][1]), "pos": v["pos"][:cnt].copy(),
                        "acc": v["acc"][:cnt].copy(), "K": v["K"][:cnt].copy(),
                        "V": v["V"][:cnt].copy(), "psi": v["psi"][:cnt].copy(),
                        "H": v["H"].copy(), "z": v["z"].copy()})
        return out

    def import_state(self, instances: Sequence[int], records, stream=None):
        inst = np.ascontiguousarray(instances, dtype=np.int32)
        buf = np.zeros(len(inst) * self.record_bytes, dtype=np.uint8)
        for i, r in enumerate(records):
            v = self._record_views(buf, i)
            cnt = int(r["count"])
            v["header"][0] = cnt
            v["header"][1] = int(r["t"])
            for name in ("pos", "acc", "K", "V", "psi"):
                v[name][:cnt] = r[name]
            v["H"][...] = r["H"]
            v["z"][...] = r["z"]
        _check(less_import_state(self.ctx, inst.ctypes.data, len(inst), buf.ctypes.data, buf.nbytes,
                                 _stream_ptr(stream)), "less_import_state")

    def read_feature_maps(self, stream=None):
        R = self.cfg.rank
        phi = np.zeros((self.instances * self.group, R), dtype=np.float32)
        psi = np.zeros((self.instances, R), dtype=np.float32)
        _check(less_read_feature_maps(self.ctx, phi.ctypes.data, psi.ctypes.data, _stream_ptr(stream)),
               "less_read_feature_maps")
        return phi, psi

    def poll_status(self, stream=None) -> int:
        return less_poll_status(self.ctx, _stream_ptr(stream))

    def kernel_variant(self, kernel: str) -> str:
        """Name of the kernel variant last launched under a KERNEL_NAMES id."""
        return less_kernel_variant(self.ctx, KERNEL_NAMES.index(kernel))

    def status_where(self) -> int:
        return less_last_status_where(self.ctx)

    def selftest_wait_timeout(self, polls: int, stream=None) -> int:
        return less_selftest_wait_timeout(self.ctx, polls, _stream_ptr(stream))

    def close(self):
        if getattr(self, "ctx", None) is not None:
            less_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def from_workload(w, weights=None, device="cuda", max_prefill_layers=1, flags=0, psi_scale=None,
                  heavy=None, recent=None, max_prompt=None) -> LessContext:
    """Context shaped like a `workloads.Workload`."""
    from . import workloads as wl
    if weights is None:
        weights = wl.make_weights(w, device)
    return LessContext(w.batch, w.layers, w.heads, w.head_dim, w.rank, w.hidden,
                       w.heavy if heavy is None else heavy, w.recent if recent is None else recent,
                       w.prompt if max_prompt is None else max_prompt, weights,
                       max_prefill_layers=max_prefill_layers, flags=flags, psi_scale=psi_scale,
                       device=device, group=getattr(w, "group", 1))
