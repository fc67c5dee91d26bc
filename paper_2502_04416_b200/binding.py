"""ctypes binding of libcmoe.so: the same calls as include/cmoe.h, argument
marshalling only.  torch is used for device memory and streams; every step of
the forward pass runs in the library's kernels.  There is no CPU fallback:
``load()`` raises if the shared library has not been built."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcmoe.so")

CMOE_BF16, CMOE_FP32 = 0, 1
GEMM_AUTO, GEMM_SIMT, GEMM_TENSOR, GEMM_TENSOR_PAIRS = 0, 1, 2, 3
N_STAGES = 5
STAGE_NAMES = ["route", "permute", "gemm1_swiglu", "gemm2_down", "combine"]

EXPORTS = [
    "cmoe_layer_create", "cmoe_hier_create", "cmoe_ffn_forward", "cmoe_ffn_forward_host", "cmoe_layer_set_gate_params",
    "cmoe_quantise_rows_fp8", "cmoe_layer_quantise_fp8",
    "cmoe_layer_get_gate_params", "cmoe_layer_update_bias", "cmoe_profile_activations", "cmoe_select_shared",
    "cmoe_cluster_update", "cmoe_cluster_distances", "cmoe_cluster_representatives", "cmoe_layer_set_gemm_path", "cmoe_layer_set_launch_chaining",
    "cmoe_layer_dims", "cmoe_get_routing", "cmoe_layer_status", "cmoe_layer_selftest_wait_timeout",
    "cmoe_layer_launch_count", "cmoe_layer_enable_stage_timing", "cmoe_layer_stage_times",
    "cmoe_layer_destroy", "cmoe_token_permute_scratch_bytes",
    "cmoe_token_permute", "cmoe_token_permute_static", "cmoe_status_string", "cmoe_last_error",
]


class CmoeConfig(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("d_ff", C.c_int32), ("n_experts", C.c_int32),
                ("n_shared", C.c_int32), ("top_k", C.c_int32), ("max_tokens", C.c_int32),
                ("dtype", C.c_int32)]


class CmoeError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        super().__init__(f"{where}: status {status} ({detail})")
        self.status = status


_lib = None


def load() -> C.CDLL:
    """Open libcmoe.so; raises if it is missing (build it with
    ``python -m paper_2502_04416_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not built; run python -m paper_2502_04416_b200.build")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.cmoe_layer_create.argtypes = [C.POINTER(CmoeConfig), vp, vp, vp, vp, vp, vp, vp, vp,
                                      C.POINTER(vp)]
    lib.cmoe_hier_create.argtypes = [i32, i32, vp, C.POINTER(vp), i32, vp, C.POINTER(vp)]
    lib.cmoe_ffn_forward.argtypes = [vp, vp, i32, vp, vp]
    lib.cmoe_ffn_forward_host.argtypes = [vp, vp, i32, vp, i32, vp]
    lib.cmoe_quantise_rows_fp8.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    lib.cmoe_layer_quantise_fp8.argtypes = [vp, vp]
    lib.cmoe_layer_set_gate_params.argtypes = [vp, vp, vp, vp]
    lib.cmoe_layer_set_gemm_path.argtypes = [vp, i32]
    lib.cmoe_layer_set_launch_chaining.argtypes = [vp, i32]
    lib.cmoe_profile_activations.argtypes = [vp, vp, i32, i32, i32, vp, i32, vp, vp]
    lib.cmoe_select_shared.argtypes = [vp, i32, i32, vp, vp]
    lib.cmoe_cluster_update.argtypes = [vp, i32, i32, vp, vp, i32, i32, vp, vp, vp]
    lib.cmoe_cluster_distances.argtypes = [vp, i32, i32, vp, i32, vp, vp, i32, vp, vp, vp]
    lib.cmoe_cluster_representatives.argtypes = [vp, vp, vp, i32, i32, vp, vp]
    lib.cmoe_layer_get_gate_params.argtypes = [vp, vp, vp, vp]
    lib.cmoe_layer_update_bias.argtypes = [vp, C.c_float, vp, vp, vp]
    lib.cmoe_layer_dims.argtypes = [vp] + [C.POINTER(i32)] * 4
    lib.cmoe_get_routing.argtypes = [vp] * 12
    lib.cmoe_layer_status.argtypes = [vp, C.POINTER(i32)]
    lib.cmoe_layer_selftest_wait_timeout.argtypes = [vp, i64, vp]
    lib.cmoe_layer_launch_count.argtypes = [vp, C.POINTER(i32)]
    lib.cmoe_layer_destroy.argtypes = [vp]
    lib.cmoe_layer_enable_stage_timing.argtypes = [vp, i32]
    lib.cmoe_layer_stage_times.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(i32)]
    lib.cmoe_token_permute_scratch_bytes.argtypes = [i32, i32]
    lib.cmoe_token_permute_scratch_bytes.restype = i64
    lib.cmoe_token_permute.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, i64, vp]
    lib.cmoe_token_permute_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.cmoe_status_string.argtypes = [C.c_int]
    lib.cmoe_status_string.restype = C.c_char_p
    lib.cmoe_last_error.restype = C.c_char_p
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int:      # default
            fn.restype = C.c_int
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != 0:
        lib = load()
        detail = lib.cmoe_status_string(status).decode() + "; " + lib.cmoe_last_error().decode()
        raise CmoeError(status, where, detail)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _stream_ptr(stream) -> Optional[int]:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return CMOE_BF16
    if t.dtype == torch.float32:
        return CMOE_FP32
    raise TypeError(f"unsupported dtype {t.dtype}")


class Layer:
    """Owns one cmoe_layer handle."""

    def __init__(self, handle: int, d_model: int, keepalive=None):
        self._h = C.c_void_p(handle)
        self.d_model = d_model
        self._keep = keepalive

    # -- construction -------------------------------------------------------
    @classmethod
    def create(cls, w_gate, w_up, w_down, neuron_perm: np.ndarray, rep_idx: np.ndarray,
               n_experts: int, n_shared: int, top_k: int, max_tokens: int,
               gate_scale_u: Optional[np.ndarray] = None,
               select_bias_b: Optional[np.ndarray] = None, stream=None) -> "Layer":
        """cmoe_layer_create.  w_gate/w_up [d_ff,d], w_down [d,d_ff]: contiguous CUDA tensors."""
        lib = load()
        for w in (w_gate, w_up, w_down):
            if not (w.is_cuda and w.is_contiguous()):
                raise ValueError("weights must be contiguous CUDA tensors")
        d_ff, d = w_gate.shape
        cfg = CmoeConfig(d, d_ff, n_experts, n_shared, top_k, max_tokens, _dtype_code(w_gate))
        perm = np.ascontiguousarray(neuron_perm, dtype=np.int32)
        rep = np.ascontiguousarray(rep_idx, dtype=np.int32)
        u = None if gate_scale_u is None else np.ascontiguousarray(gate_scale_u, dtype=np.float32)
        b = None if select_bias_b is None else np.ascontiguousarray(select_bias_b, dtype=np.float32)
        out = C.c_void_p()
        st = lib.cmoe_layer_create(C.byref(cfg), w_gate.data_ptr(), w_up.data_ptr(),
                                   w_down.data_ptr(), _np_ptr(perm), _np_ptr(rep), _np_ptr(u),
                                   _np_ptr(b), _stream_ptr(stream), C.byref(out))
        _check(st, "cmoe_layer_create")
        return cls(out.value, d)

    @classmethod
    def create_hier(cls, w_router, inner: Sequence["Layer"], outer_top_k: int, max_tokens: int,
                    stream=None) -> "Layer":
        """cmoe_hier_create; the inner layers are consumed."""
        lib = load()
        n = len(inner)
        arr = (C.c_void_p * n)(*[l._h.value for l in inner])
        out = C.c_void_p()
        st = lib.cmoe_hier_create(n, outer_top_k, w_router.data_ptr(), arr, max_tokens,
                                  _stream_ptr(stream), C.byref(out))
        _check(st, "cmoe_hier_create")
        for l in inner:
            l._h = C.c_void_p(None)
        return cls(out.value, inner[0].d_model)

    # -- forward ------------------------------------------------------------
    def forward(self, x, out=None, stream=None):
        """cmoe_ffn_forward: x [T,d] CUDA tensor -> out [T,d]."""
        import torch
        if out is None:
            out = torch.empty_like(x)
        st = load().cmoe_ffn_forward(self._h, x.data_ptr(), x.shape[0], out.data_ptr(),
                                     _stream_ptr(stream))
        _check(st, "cmoe_ffn_forward")
        return out

    def forward_host(self, x_host, out_host, chunk_tokens: int = 0, stream=None):
        """cmoe_ffn_forward_host: x_host / out_host are CPU tensors [T,d] (pinned for overlap);
        asynchronous on the stream, out_host is complete once the stream has passed the call."""
        if x_host.is_cuda or out_host.is_cuda or not (x_host.is_contiguous() and out_host.is_contiguous()):
            raise ValueError("forward_host takes contiguous CPU tensors")
        st = load().cmoe_ffn_forward_host(self._h, x_host.data_ptr(), x_host.shape[0], out_host.data_ptr(),
                                          chunk_tokens, _stream_ptr(stream))
        _check(st, "cmoe_ffn_forward_host")
        return out_host

    def quantise_fp8(self, stream=None) -> None:
        """cmoe_layer_quantise_fp8: FP8 (E4M3, power-of-two scale per output channel) expert weights."""
        _check(load().cmoe_layer_quantise_fp8(self._h, _stream_ptr(stream)), "cmoe_layer_quantise_fp8")

    def set_gate_params(self, gate_scale_u=None, select_bias_b=None, stream=None) -> None:
        u = None if gate_scale_u is None else np.ascontiguousarray(gate_scale_u, dtype=np.float32)
        b = None if select_bias_b is None else np.ascontiguousarray(select_bias_b, dtype=np.float32)
        _check(load().cmoe_layer_set_gate_params(self._h, _np_ptr(u), _np_ptr(b),
                                                 _stream_ptr(stream)), "cmoe_layer_set_gate_params")

    def get_gate_params(self, stream=None):
        """(gate_scale_u, select_bias_b) as float32 arrays of length n_routed_groups."""
        n = self.dims()["n_routed_groups"]
        u, b = np.zeros(n, np.float32), np.zeros(n, np.float32)
        _check(load().cmoe_layer_get_gate_params(self._h, _np_ptr(u), _np_ptr(b), _stream_ptr(stream)),
               "cmoe_layer_get_gate_params")
        return u, b

    def update_bias(self, gamma: float = 1e-3, target_share=None, want_utilisation: bool = True, stream=None):
        """cmoe_layer_update_bias: one load-balancing step from the last forward's counts.
        Returns the utilisation p_i (float32 [n_routed_groups]) or None."""
        n = self.dims()["n_routed_groups"]
        tgt = None if target_share is None else np.ascontiguousarray(target_share, dtype=np.float32)
        util = np.zeros(n, np.float32) if want_utilisation else None
        _check(load().cmoe_layer_update_bias(self._h, gamma, _np_ptr(tgt), _np_ptr(util),
                                             _stream_ptr(stream)), "cmoe_layer_update_bias")
        return util

    def profile_activations(self, x, k_a: int, act_bits, act_count, token0: int = 0, stream=None) -> None:
        """cmoe_profile_activations on CUDA tensors: x [n, d_model] in the layer's dtype, act_bits
        int32/uint32-sized [d_ff, words], act_count int32 [d_ff]; both accumulate."""
        _check(load().cmoe_profile_activations(self._h, x.data_ptr(), x.shape[0], k_a, token0, act_bits.data_ptr(),
                                               act_bits.shape[1], act_count.data_ptr(), _stream_ptr(stream)),
               "cmoe_profile_activations")

    def set_gemm_path(self, path: int) -> None:
        _check(load().cmoe_layer_set_gemm_path(self._h, path), "cmoe_layer_set_gemm_path")

    def set_launch_chaining(self, on: bool) -> None:
        _check(load().cmoe_layer_set_launch_chaining(self._h, 1 if on else 0), "cmoe_layer_set_launch_chaining")

    def dims(self) -> Dict[str, int]:
        v = [C.c_int32() for _ in range(4)]
        _check(load().cmoe_layer_dims(self._h, *[C.byref(a) for a in v]), "cmoe_layer_dims")
        return dict(n_routed_groups=v[0].value, top_k=v[1].value, n_outer=v[2].value,
                    outer_top_k=v[3].value)

    def routing(self, n_tokens: int, n_routed_per_layer: int) -> Dict[str, np.ndarray]:
        """cmoe_get_routing for the last forward of ``n_tokens`` tokens."""
        dm = self.dims()
        ok = dm["outer_top_k"]
        R = n_tokens * (ok if ok else 1)
        k, G, nr = dm["top_k"], dm["n_routed_groups"], n_routed_per_layer
        r = dict(keys=np.zeros((R, nr), np.float32), scores=np.zeros((R, nr), np.float32),
                 topk_idx=np.zeros((R, k), np.int32), topk_gate=np.zeros((R, k), np.float32),
                 counts=np.zeros(G, np.int32), offsets=np.zeros(G + 1, np.int32),
                 row_token=np.zeros(R * k, np.int32), row_of=np.zeros((R, k), np.int32))
        if ok:
            r.update(outer_idx=np.zeros((n_tokens, ok), np.int32),
                     outer_w=np.zeros((n_tokens, ok), np.float32),
                     outer_row_token=np.zeros(R, np.int32))
        order = ["keys", "scores", "topk_idx", "topk_gate", "counts", "offsets", "row_token",
                 "row_of", "outer_idx", "outer_w", "outer_row_token"]
        _check(load().cmoe_get_routing(self._h, *[_np_ptr(r.get(n)) for n in order]),
               "cmoe_get_routing")
        return r

    def status(self) -> int:
        """Device error word of the last forward (0 = none).  A non-zero word is reported once:
        the call also clears it and the layer's K-slice tickets."""
        w = C.c_int32()
        st = load().cmoe_layer_status(self._h, C.byref(w))
        if st not in (0, -6):
            _check(st, "cmoe_layer_status")
        return w.value

    def selftest_wait_timeout(self, limit_cycles: int = 2_000_000, stream=None) -> None:
        """cmoe_layer_selftest_wait_timeout: one warp runs a bounded wait to its limit."""
        _check(load().cmoe_layer_selftest_wait_timeout(self._h, limit_cycles, _stream_ptr(stream)),
               "cmoe_layer_selftest_wait_timeout")

    def launch_count(self) -> int:
        w = C.c_int32()
        _check(load().cmoe_layer_launch_count(self._h, C.byref(w)), "cmoe_layer_launch_count")
        return w.value

    def enable_stage_timing(self, ring_steps: int) -> None:
        _check(load().cmoe_layer_enable_stage_timing(self._h, ring_steps),
               "cmoe_layer_enable_stage_timing")

    def stage_times(self):
        """(per-stage summed milliseconds [N_STAGES], forwards covered)."""
        ms = (C.c_float * N_STAGES)()
        n = C.c_int32()
        _check(load().cmoe_layer_stage_times(self._h, ms, C.byref(n)), "cmoe_layer_stage_times")
        return [float(v) for v in ms], n.value

    def destroy(self) -> None:
        if self._h and self._h.value:
            load().cmoe_layer_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def quantise_rows_fp8(w, want_dequantised: bool = False, stream=None):
    """cmoe_quantise_rows_fp8 on a CUDA bf16 tensor [rows, cols]: (codes uint8, scale float32[, dequantised bf16])."""
    import torch
    rows, cols = w.shape
    codes = torch.empty((rows, cols), dtype=torch.uint8, device=w.device)
    scale = torch.empty(rows, dtype=torch.float32, device=w.device)
    deq = torch.empty_like(w) if want_dequantised else None
    _check(load().cmoe_quantise_rows_fp8(w.data_ptr(), rows, cols, codes.data_ptr(), scale.data_ptr(),
                                         deq.data_ptr() if deq is not None else None, _stream_ptr(stream)),
           "cmoe_quantise_rows_fp8")
    return (codes, scale, deq) if want_dequantised else (codes, scale)


def token_permute_scratch_bytes(n_rows: int, n_groups: int) -> int:
    return int(load().cmoe_token_permute_scratch_bytes(n_rows, n_groups))


def token_permute(topk_idx, n_groups: int, stream=None):
    """cmoe_token_permute on a CUDA int32 tensor [n_rows, n_k].
    Returns (counts, offsets, row_token, row_of) CUDA int32 tensors."""
    import torch
    n_rows, n_k = topk_idx.shape
    dev = topk_idx.device
    counts = torch.empty(n_groups, dtype=torch.int32, device=dev)
    offsets = torch.empty(n_groups + 1, dtype=torch.int32, device=dev)
    row_token = torch.empty(max(n_rows * n_k, 1), dtype=torch.int32, device=dev)
    row_of = torch.empty((n_rows, n_k), dtype=torch.int32, device=dev)
    nbytes = token_permute_scratch_bytes(n_rows, n_groups)
    scratch = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
    st = load().cmoe_token_permute(topk_idx.data_ptr(), n_rows, n_k, n_groups, counts.data_ptr(),
                                   offsets.data_ptr(), row_token.data_ptr(), row_of.data_ptr(),
                                   scratch.data_ptr(), nbytes, _stream_ptr(stream))
    _check(st, "cmoe_token_permute")
    return counts, offsets, row_token[:n_rows * n_k], row_of


def select_shared(act_count, n_select: int, stream=None):
    """cmoe_select_shared on a CUDA int32 tensor [d_ff]; returns a CUDA int32 tensor [n_select]."""
    import torch
    out = torch.empty(max(n_select, 1), dtype=torch.int32, device=act_count.device)
    _check(load().cmoe_select_shared(act_count.data_ptr(), act_count.shape[0], n_select, out.data_ptr(),
                                     _stream_ptr(stream)), "cmoe_select_shared")
    return out[:n_select]


def cluster_update(act_bits, n_tokens: int, neuron_idx, assign, centroid_count, cluster_size, stream=None) -> None:
    """cmoe_cluster_update on CUDA tensors (act_bits [d_ff, words] 32-bit, neuron_idx / assign int32 [n],
    centroid_count int32 [n_clusters, n_tokens], cluster_size int32 [n_clusters]; both updated in place)."""
    _check(load().cmoe_cluster_update(act_bits.data_ptr(), act_bits.shape[1], n_tokens, neuron_idx.data_ptr(),
                                      assign.data_ptr(), neuron_idx.shape[0], centroid_count.shape[0],
                                      centroid_count.data_ptr(), cluster_size.data_ptr(), _stream_ptr(stream)),
           "cmoe_cluster_update")


def cluster_distances(act_bits, n_tokens: int, neuron_idx, centroid_count, cluster_size, stream=None):
    """cmoe_cluster_distances; returns the CUDA int64 tensor [n, n_clusters] of size_j^2 * d_ij^2."""
    import torch
    n, c = neuron_idx.shape[0], centroid_count.shape[0]
    sqnorm = torch.empty(c, dtype=torch.int64, device=act_bits.device)
    out = torch.empty((max(n, 1), c), dtype=torch.int64, device=act_bits.device)
    _check(load().cmoe_cluster_distances(act_bits.data_ptr(), act_bits.shape[1], n_tokens, neuron_idx.data_ptr(), n,
                                         centroid_count.data_ptr(), cluster_size.data_ptr(), c, sqnorm.data_ptr(),
                                         out.data_ptr(), _stream_ptr(stream)), "cmoe_cluster_distances")
    return out[:n]


def cluster_representatives(scaled_sq_dist, neuron_idx, assign, stream=None):
    """cmoe_cluster_representatives; returns a CUDA int32 tensor [n_clusters]."""
    import torch
    c = scaled_sq_dist.shape[1]
    out = torch.empty(c, dtype=torch.int32, device=scaled_sq_dist.device)
    _check(load().cmoe_cluster_representatives(scaled_sq_dist.data_ptr(), neuron_idx.data_ptr(), assign.data_ptr(),
                                               neuron_idx.shape[0], c, out.data_ptr(), _stream_ptr(stream)),
           "cmoe_cluster_representatives")
    return out


STATIC_PERMUTE_MAX_CELLS = 262144


def token_permute_static(topk_idx, n_groups: int, out=None, stream=None):
    """cmoe_token_permute_static: the same permutation, for callers that may not allocate
    device memory.  The library's built-in 1 MiB scratch array replaces the scratch buffer;
    pass ``out`` = (counts, offsets, row_token, row_of) preallocated CUDA int32 tensors to
    keep the call itself free of allocations (this wrapper allocates them otherwise).
    Calls on one device share that array and must not overlap on the GPU."""
    import torch
    n_rows, n_k = topk_idx.shape
    dev = topk_idx.device
    if out is None:
        out = (torch.empty(n_groups, dtype=torch.int32, device=dev),
               torch.empty(n_groups + 1, dtype=torch.int32, device=dev),
               torch.empty(max(n_rows * n_k, 1), dtype=torch.int32, device=dev),
               torch.empty((n_rows, n_k), dtype=torch.int32, device=dev))
    counts, offsets, row_token, row_of = out
    st = load().cmoe_token_permute_static(topk_idx.data_ptr(), n_rows, n_k, n_groups,
                                          counts.data_ptr(), offsets.data_ptr(),
                                          row_token.data_ptr(), row_of.data_ptr(),
                                          _stream_ptr(stream))
    _check(st, "cmoe_token_permute_static")
    return counts, offsets, row_token[:n_rows * n_k], row_of
