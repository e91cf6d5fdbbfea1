"""ctypes binding of libroco's C ABI (argument marshalling only; every step runs in the CUDA kernels).

PyTorch is used for device memory and streams.  There is no CPU path: loading fails loudly when the
compiled library is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libroco.so")

ROCO_OK = 0
ROCO_F32, ROCO_BF16 = 0, 1
ROCO_SCOPE_EXCLUDE_TOP_R, ROCO_SCOPE_LOWEST_R = 0, 1
ROCO_EVICT_FIRST, ROCO_ATTEND_FIRST = 0, 1
(ROCO_POLICY_ROCO, ROCO_POLICY_RANDOM, ROCO_POLICY_RECENCY, ROCO_POLICY_STREAMLLM, ROCO_POLICY_SCISSORHANDS,
 ROCO_POLICY_H2O, ROCO_POLICY_TOVA, ROCO_POLICY_MAS_WINDOW) = range(8)

EXPORTS = ("roco_version", "roco_status_string", "roco_prefill_workspace_bytes", "roco_prefill",
           "roco_prefill_uses_tensor_cores", "roco_prefill_static", "roco_prefill_workspace_bytes_lowest_r",
           "roco_block_step", "roco_gqa_decode_step", "roco_decode_step_policy",
           "roco_decode_split_workspace_bytes", "roco_decode_step_split", "roco_prefill_blockwise",
           "roco_decode_step", "roco_decode_host_staging_bytes", "roco_decode_step_host", "roco_device_status",
           "roco_prefill_attend_workspace_bytes", "roco_prefill_attend", "roco_selftest_wait_timeout",
           "roco_consistency_step", "roco_selftest_read_stream", "roco_decode_host_pipeline_staging_bytes",
           "roco_decode_step_host_begin", "roco_decode_step_host_end", "roco_gqa_block_step",
           "roco_prefill_blockwise_gqa", "roco_prefill_with_output", "roco_decode_cluster_ranks",
           "roco_decode_step_cluster", "roco_decode_step_policy_ordered", "roco_decode_step_split_ordered")


class RocoError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: status {code} ({status_string(code)})")
        self.code = code


class roco_cache(C.Structure):
    _fields_ = [("kv_dtype", C.c_int32), ("S", C.c_int32), ("G", C.c_int32), ("d", C.c_int32), ("B", C.c_int32),
                ("K", C.c_void_p), ("V", C.c_void_p), ("s", C.c_void_p), ("q", C.c_void_p),
                ("n", C.c_void_p), ("pos", C.c_void_p), ("live", C.c_void_p), ("t_next", C.c_void_p),
                ("status", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2402_06262_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        L.roco_version.restype = C.c_int
        L.roco_status_string.restype = C.c_char_p
        L.roco_status_string.argtypes = [C.c_int]
        L.roco_prefill_workspace_bytes.restype = C.c_size_t
        L.roco_prefill_workspace_bytes.argtypes = [C.POINTER(roco_cache), C.c_int]
        L.roco_prefill_workspace_bytes_lowest_r.restype = C.c_size_t
        L.roco_prefill_workspace_bytes_lowest_r.argtypes = [C.POINTER(roco_cache), C.c_int]
        L.roco_prefill_uses_tensor_cores.restype = C.c_int
        L.roco_prefill_uses_tensor_cores.argtypes = [C.POINTER(roco_cache)]
        L.roco_decode_host_staging_bytes.restype = C.c_size_t
        L.roco_decode_host_staging_bytes.argtypes = [C.POINTER(roco_cache)]
        L.roco_prefill.restype = C.c_int
        L.roco_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                   C.c_int, C.c_float, C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p]
        L.roco_prefill_with_output.restype = C.c_int
        L.roco_prefill_with_output.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                               C.c_int, C.c_int, C.c_int, C.c_float, C.POINTER(roco_cache), C.c_void_p,
                                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.roco_prefill_static.restype = C.c_int
        L.roco_prefill_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                          C.c_int, C.c_int, C.c_float, C.POINTER(roco_cache), C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p]
        L.roco_prefill_attend_workspace_bytes.restype = C.c_size_t
        L.roco_prefill_attend_workspace_bytes.argtypes = [C.POINTER(roco_cache)]
        L.roco_prefill_attend.restype = C.c_int
        L.roco_prefill_attend.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                          C.c_void_p]
        L.roco_decode_step.restype = C.c_int
        L.roco_decode_step.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                       C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        for fn in (L.roco_block_step, L.roco_gqa_decode_step):
            fn.restype = C.c_int
            fn.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                           C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.roco_gqa_block_step.restype = C.c_int
        L.roco_gqa_block_step.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                          C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p]
        L.roco_prefill_blockwise_gqa.restype = C.c_int
        L.roco_prefill_blockwise_gqa.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                                 C.c_int, C.c_int, C.c_float, C.POINTER(roco_cache), C.c_void_p,
                                                 C.c_void_p, C.c_void_p]
        L.roco_prefill_blockwise.restype = C.c_int
        L.roco_prefill_blockwise.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                             C.c_float, C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p]
        L.roco_decode_split_workspace_bytes.restype = C.c_size_t
        L.roco_decode_split_workspace_bytes.argtypes = [C.POINTER(roco_cache), C.c_int]
        L.roco_decode_step_split_ordered.restype = C.c_int
        L.roco_decode_step_split_ordered.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                                     C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.roco_decode_step_split.restype = C.c_int
        L.roco_decode_step_split.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                             C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.roco_decode_cluster_ranks.restype = C.c_int
        L.roco_decode_cluster_ranks.argtypes = [C.POINTER(roco_cache)]
        L.roco_decode_step_cluster.restype = C.c_int
        L.roco_decode_step_cluster.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                               C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_void_p, C.c_void_p]
        L.roco_decode_step_policy_ordered.restype = C.c_int
        L.roco_decode_step_policy_ordered.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p,
                                                      C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_float, C.c_void_p,
                                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.roco_decode_step_policy.restype = C.c_int
        L.roco_decode_step_policy.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                              C.c_int, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                              C.c_void_p, C.c_void_p]
        L.roco_decode_step_host.restype = C.c_int
        L.roco_decode_step_host.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                            C.c_int, C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_size_t, C.c_void_p]
        L.roco_consistency_step.restype = C.c_int
        L.roco_consistency_step.argtypes = [C.POINTER(roco_cache), C.POINTER(roco_cache), C.c_int, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p]
        L.roco_decode_host_pipeline_staging_bytes.restype = C.c_size_t
        L.roco_decode_host_pipeline_staging_bytes.argtypes = [C.POINTER(roco_cache)]
        L.roco_decode_step_host_begin.restype = C.c_int
        L.roco_decode_step_host_begin.argtypes = L.roco_decode_step_host.argtypes
        L.roco_decode_step_host_end.restype = C.c_int
        L.roco_decode_step_host_end.argtypes = []
        L.roco_selftest_read_stream.restype = C.c_int
        L.roco_selftest_read_stream.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.roco_selftest_wait_timeout.restype = C.c_int
        L.roco_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.roco_device_status.restype = C.c_int
        L.roco_device_status.argtypes = [C.POINTER(roco_cache), C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().roco_status_string(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Cache:
    """Device tensors of the budgeted cache for S sequences x G units, plus the C struct over them."""

    def __init__(self, S: int, G: int, B: int, d: int, dtype: torch.dtype, device="cuda"):
        assert dtype in (torch.float32, torch.bfloat16)
        self.S, self.G, self.B, self.d, self.dtype = S, G, B, d, dtype
        self.K = torch.zeros(S, G, B, d, dtype=dtype, device=device)
        self.V = torch.zeros(S, G, B, d, dtype=dtype, device=device)
        self.s = torch.zeros(S, G, B, dtype=torch.float32, device=device)
        self.q = torch.zeros(S, G, B, dtype=torch.float32, device=device)
        self.n = torch.zeros(S, G, B, dtype=torch.int32, device=device)
        self.pos = torch.full((S, G, B), -1, dtype=torch.int32, device=device)
        self.live = torch.zeros(S, G, dtype=torch.int32, device=device)
        self.t_next = torch.zeros(S, G, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.c = roco_cache(ROCO_F32 if dtype == torch.float32 else ROCO_BF16, S, G, d, B,
                            self.K.data_ptr(), self.V.data_ptr(), self.s.data_ptr(), self.q.data_ptr(),
                            self.n.data_ptr(), self.pos.data_ptr(), self.live.data_ptr(), self.t_next.data_ptr(),
                            self.status.data_ptr())

    @property
    def U(self) -> int:
        return self.S * self.G


def roco_prefill_workspace_bytes(cache: Cache, Lmax: int) -> int:
    return int(lib().roco_prefill_workspace_bytes(C.byref(cache.c), Lmax))


def roco_prefill_workspace_bytes_lowest_r(cache: Cache, Lmax: int) -> int:
    return int(lib().roco_prefill_workspace_bytes_lowest_r(C.byref(cache.c), Lmax))


def roco_prefill_uses_tensor_cores(cache: Cache) -> bool:
    return bool(lib().roco_prefill_uses_tensor_cores(C.byref(cache.c)))


def roco_prefill(Q, K, V, lens: Sequence[int], B: int, r: int, cache: Cache, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R,
                 count_self=1, scale: Optional[float] = None, lse_out=None, s_full=None, q_full=None,
                 workspace: Optional[torch.Tensor] = None, attn_out=None):
    """Q, K, V: [S][G][Lmax][d] device tensors.  Fills `cache`.  attn_out ([S][G][Lmax][d]): also the prompt's
    causal attention output (roco_prefill_with_output)."""
    Lmax = Q.shape[2]
    scale = cache.d ** -0.5 if scale is None else scale
    if workspace is None:
        nbytes = (roco_prefill_workspace_bytes_lowest_r if scope_mode == ROCO_SCOPE_LOWEST_R
                  else roco_prefill_workspace_bytes)(cache, Lmax)
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=Q.device)
    lens_arr = (C.c_int32 * len(lens))(*[int(x) for x in lens])
    if attn_out is not None:
        rc = lib().roco_prefill_with_output(_ptr(Q), _ptr(K), _ptr(V), C.cast(lens_arr, C.c_void_p), Lmax, B, r,
                                            scope_mode, count_self, scale, C.byref(cache.c), _ptr(lse_out),
                                            _ptr(s_full), _ptr(q_full), _ptr(attn_out), _ptr(workspace),
                                            workspace.numel(), _stream())
    else:
        rc = lib().roco_prefill(_ptr(Q), _ptr(K), _ptr(V), C.cast(lens_arr, C.c_void_p), Lmax, B, r, scope_mode,
                                count_self, scale, C.byref(cache.c), _ptr(lse_out), _ptr(s_full), _ptr(q_full),
                                _ptr(workspace), workspace.numel(), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_prefill")
    return workspace


PREFILL_STATIC_SCRATCH_BYTES = 8 << 20


def roco_prefill_static(Q, K, V, lens: Sequence[int], B: int, r: int, cache: Cache,
                        scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R, count_self=1, scale: Optional[float] = None,
                        lse_out=None, s_full=None, q_full=None):
    """roco_prefill for callers that cannot allocate a workspace: the scratch is an 8 MiB array built into the
    library (so S*G*Lmax is limited; larger problems raise RocoError with the workspace status).  Calls on one
    device share that array: keep them on one stream."""
    Lmax = Q.shape[2]
    scale = cache.d ** -0.5 if scale is None else scale
    lens_arr = (C.c_int32 * len(lens))(*[int(x) for x in lens])
    rc = lib().roco_prefill_static(_ptr(Q), _ptr(K), _ptr(V), C.cast(lens_arr, C.c_void_p), Lmax, B, r, scope_mode,
                                   count_self, scale, C.byref(cache.c), _ptr(lse_out), _ptr(s_full), _ptr(q_full),
                                   _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_prefill_static")


def roco_prefill_attend_workspace_bytes(cache: Cache) -> int:
    return int(lib().roco_prefill_attend_workspace_bytes(C.byref(cache.c)))


def roco_prefill_attend(cache: Cache, Q, K, V, lens: Sequence[int], lse, attn_out, scale: Optional[float] = None,
                        workspace: Optional[torch.Tensor] = None):
    """Causal attention output of the prompt pass from the row log-sum-exp `lse` that roco_prefill returned.
    Q, K, V, attn_out: [S][G][Lmax][d] bf16 device tensors (d = 128); lse: [S][G][Lmax] fp32."""
    Lmax = Q.shape[2]
    scale = cache.d ** -0.5 if scale is None else scale
    if workspace is None:
        workspace = torch.empty(roco_prefill_attend_workspace_bytes(cache), dtype=torch.uint8, device=Q.device)
    lens_arr = (C.c_int32 * len(lens))(*[int(x) for x in lens])
    rc = lib().roco_prefill_attend(C.byref(cache.c), _ptr(Q), _ptr(K), _ptr(V), C.cast(lens_arr, C.c_void_p), Lmax,
                                   scale, _ptr(lse), _ptr(attn_out), _ptr(workspace), workspace.numel(), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_prefill_attend")
    return workspace


def roco_selftest_read_stream(buf: torch.Tensor, sink: Optional[torch.Tensor] = None):
    """One launch that reads every byte of `buf` (device tensor) with plain 16-byte loads; time it to get the
    device's read-only streaming rate.  sink: int64 [1] device checksum accumulator, or None."""
    rc = lib().roco_selftest_read_stream(_ptr(buf), buf.numel() * buf.element_size(), _ptr(sink), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_selftest_read_stream")


def roco_selftest_wait_timeout(status: torch.Tensor, waited_ms: Optional[torch.Tensor] = None):
    """Launches the bounded-wait self-test: `status` (int32 [1], device) gets ROCO_DEV_WAIT_TIMEOUT once the
    kernel's wait has run out (about two seconds); `waited_ms` (int32 [1], device) how long that took."""
    rc = lib().roco_selftest_wait_timeout(_ptr(status), _ptr(waited_ms), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_selftest_wait_timeout")


def roco_decode_step(cache: Cache, q, k_new, v_new, r: int, attn_out, evicted_slot, evicted_pos=None, lse_out=None,
                     scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R, step_order=ROCO_EVICT_FIRST, scale: Optional[float] = None):
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_decode_step(C.byref(cache.c), _ptr(q), _ptr(k_new), _ptr(v_new), r, scope_mode, step_order,
                                scale, _ptr(attn_out), _ptr(lse_out), _ptr(evicted_slot), _ptr(evicted_pos), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step")


def roco_prefill_blockwise(Q, K, V, lens: Sequence[int], b: int, r: int, cache: Cache, attn_out, evicted_slot,
                           scale: Optional[float] = None):
    """Encode the prompts block by block (b tokens per evict-and-encode step) through the budgeted cache."""
    scale = cache.d ** -0.5 if scale is None else scale
    lens_arr = (C.c_int32 * len(lens))(*[int(x) for x in lens])
    rc = lib().roco_prefill_blockwise(_ptr(Q), _ptr(K), _ptr(V), C.cast(lens_arr, C.c_void_p), int(Q.shape[2]), b, r,
                                      scale, C.byref(cache.c), _ptr(attn_out), _ptr(evicted_slot), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_prefill_blockwise")


def roco_decode_split_workspace_bytes(cache: Cache, splits: int) -> int:
    return int(lib().roco_decode_split_workspace_bytes(C.byref(cache.c), splits))


def roco_decode_step_split(cache: Cache, q, k_new, v_new, r: int, splits: int, attn_out, evicted_slot, workspace,
                           evicted_pos=None, lse_out=None, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R,
                           scale: Optional[float] = None, step_order: Optional[int] = None):
    """roco_decode_step with every unit's slots divided among `splits` CTAs.  step_order None: the entry point with
    the order of Fig. 1 (evict, insert, attend); else roco_decode_step_split_ordered."""
    scale = cache.d ** -0.5 if scale is None else scale
    if step_order is None:
        rc = lib().roco_decode_step_split(C.byref(cache.c), _ptr(q), _ptr(k_new), _ptr(v_new), r, scope_mode, splits,
                                          scale, _ptr(attn_out), _ptr(lse_out), _ptr(evicted_slot),
                                          _ptr(evicted_pos), _ptr(workspace), workspace.numel(), _stream())
    else:
        rc = lib().roco_decode_step_split_ordered(C.byref(cache.c), _ptr(q), _ptr(k_new), _ptr(v_new), r, scope_mode,
                                                  step_order, splits, scale, _ptr(attn_out), _ptr(lse_out),
                                                  _ptr(evicted_slot), _ptr(evicted_pos), _ptr(workspace),
                                                  workspace.numel(), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step_split")


def roco_decode_cluster_ranks(cache: Cache) -> int:
    """CTAs per unit that suit this cache's shape on the current device (1: one CTA per unit)."""
    return int(lib().roco_decode_cluster_ranks(C.byref(cache.c)))


def roco_decode_step_cluster(cache: Cache, q, k_new, v_new, r: int, attn_out, evicted_slot, evicted_pos=None,
                             lse_out=None, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R, step_order=ROCO_EVICT_FIRST,
                             ranks: int = 0, scale: Optional[float] = None):
    """roco_decode_step with a cluster of `ranks` CTAs per unit (0: chosen from the shape; 1: one CTA per unit)."""
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_decode_step_cluster(C.byref(cache.c), _ptr(q), _ptr(k_new), _ptr(v_new), r, scope_mode,
                                        step_order, ranks, scale, _ptr(attn_out), _ptr(lse_out), _ptr(evicted_slot),
                                        _ptr(evicted_pos), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step_cluster")


def roco_decode_step_policy(cache: Cache, q, k_new, v_new, policy: int, r: int, attn_out, evicted_slot,
                            evicted_pos=None, lse_out=None, rnd=None, scale: Optional[float] = None,
                            step_order: Optional[int] = None):
    """Decode step under one of the Table 1 policies; rnd: [S][G] int32/uint32 draws.  step_order None: the entry
    point with the order of Fig. 1 (evict, insert, attend); else roco_decode_step_policy_ordered."""
    scale = cache.d ** -0.5 if scale is None else scale
    if step_order is None:
        rc = lib().roco_decode_step_policy(C.byref(cache.c), _ptr(q), _ptr(k_new), _ptr(v_new), policy, r, _ptr(rnd),
                                           scale, _ptr(attn_out), _ptr(lse_out), _ptr(evicted_slot),
                                           _ptr(evicted_pos), _stream())
    else:
        rc = lib().roco_decode_step_policy_ordered(C.byref(cache.c), _ptr(q), _ptr(k_new), _ptr(v_new), policy, r,
                                                   step_order, _ptr(rnd), scale, _ptr(attn_out), _ptr(lse_out),
                                                   _ptr(evicted_slot), _ptr(evicted_pos), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step_policy")


def roco_block_step(cache: Cache, Q, K_new, V_new, r: int, attn_out, evicted_slot, evicted_pos=None, lse_out=None,
                    scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R, scale: Optional[float] = None):
    """Block-wise evict-and-encode of b = Q.shape[2] tokens per unit.  Q, K_new, V_new: [S][G][b][d]."""
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_block_step(C.byref(cache.c), _ptr(Q), _ptr(K_new), _ptr(V_new), int(Q.shape[2]), r, scope_mode,
                               scale, _ptr(attn_out), _ptr(lse_out), _ptr(evicted_slot), _ptr(evicted_pos), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_block_step")


def roco_gqa_block_step(cache: Cache, Q, K_new, V_new, r: int, attn_out, evicted_slot, evicted_pos=None,
                        lse_out=None, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R, scale: Optional[float] = None):
    """Block-wise evict-and-encode of b = Q.shape[2] tokens per key-value head shared by group = Q.shape[3] query
    heads.  Q: [S][G][b][group][d]; K_new, V_new: [S][G][b][d]."""
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_gqa_block_step(C.byref(cache.c), _ptr(Q), _ptr(K_new), _ptr(V_new), int(Q.shape[2]),
                                   int(Q.shape[3]), r, scope_mode, scale, _ptr(attn_out), _ptr(lse_out),
                                   _ptr(evicted_slot), _ptr(evicted_pos), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_gqa_block_step")


def roco_prefill_blockwise_gqa(Q, K, V, lens: Sequence[int], b: int, r: int, cache: Cache, attn_out, evicted_slot,
                               scale: Optional[float] = None):
    """roco_prefill_blockwise for a grouped-query model.  Q, attn_out: [S][G][Lmax][group][d]; K, V: [S][G][Lmax][d]."""
    scale = cache.d ** -0.5 if scale is None else scale
    lens_arr = (C.c_int32 * len(lens))(*[int(x) for x in lens])
    rc = lib().roco_prefill_blockwise_gqa(_ptr(Q), _ptr(K), _ptr(V), C.cast(lens_arr, C.c_void_p), int(K.shape[2]), b,
                                          int(Q.shape[3]), r, scale, C.byref(cache.c), _ptr(attn_out),
                                          _ptr(evicted_slot), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_prefill_blockwise_gqa")


def roco_gqa_decode_step(cache: Cache, Q, k_new, v_new, r: int, attn_out, evicted_slot, evicted_pos=None,
                         lse_out=None, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R, scale: Optional[float] = None):
    """Decode step of key-value heads shared by group = Q.shape[2] query heads.  Q: [S][G][group][d]."""
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_gqa_decode_step(C.byref(cache.c), _ptr(Q), _ptr(k_new), _ptr(v_new), int(Q.shape[2]), r,
                                    scope_mode, scale, _ptr(attn_out), _ptr(lse_out), _ptr(evicted_slot),
                                    _ptr(evicted_pos), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_gqa_decode_step")


def roco_consistency_step(full: Cache, budgeted: Cache, policy: int, overlap, jaccard_sum, samples):
    """Overlap of the budgeted cache's retained tokens with the full cache's top-B by the policy's score, per unit
    (overlap [S][G] int32), accumulated as Jaccard similarity into jaccard_sum [S][G] fp32 / samples [S][G] int32."""
    rc = lib().roco_consistency_step(C.byref(full.c), C.byref(budgeted.c), policy, _ptr(overlap), _ptr(jaccard_sum),
                                     _ptr(samples), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_consistency_step")


def roco_decode_host_staging_bytes(cache: Cache) -> int:
    return int(lib().roco_decode_host_staging_bytes(C.byref(cache.c)))


def roco_decode_step_host(cache: Cache, q_host, k_new_host, v_new_host, r: int, attn_out_host, evicted_slot_host,
                          evicted_pos_host, staging, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R,
                          step_order=ROCO_EVICT_FIRST, scale: Optional[float] = None):
    """Same step with host (pinned) per-step tensors; synchronises the stream."""
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_decode_step_host(C.byref(cache.c), _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), r,
                                     scope_mode, step_order, scale, _ptr(attn_out_host), _ptr(evicted_slot_host),
                                     _ptr(evicted_pos_host), _ptr(staging), staging.numel(), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step_host")


def roco_decode_host_pipeline_staging_bytes(cache: Cache) -> int:
    return int(lib().roco_decode_host_pipeline_staging_bytes(C.byref(cache.c)))


def roco_decode_step_host_begin(cache: Cache, q_host, k_new_host, v_new_host, r: int, attn_out_host,
                                evicted_slot_host, evicted_pos_host, staging, scope_mode=ROCO_SCOPE_EXCLUDE_TOP_R,
                                step_order=ROCO_EVICT_FIRST, scale: Optional[float] = None):
    """First half of the host-buffer step: enqueues copies in, kernel, copies out; does not wait."""
    scale = cache.d ** -0.5 if scale is None else scale
    rc = lib().roco_decode_step_host_begin(C.byref(cache.c), _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), r,
                                           scope_mode, step_order, scale, _ptr(attn_out_host),
                                           _ptr(evicted_slot_host), _ptr(evicted_pos_host), _ptr(staging),
                                           staging.numel(), _stream())
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step_host_begin")


def roco_decode_step_host_end():
    """Second half: waits until the oldest begun step's results are in its host buffers."""
    rc = lib().roco_decode_step_host_end()
    if rc != ROCO_OK:
        raise RocoError(rc, "roco_decode_step_host_end")


def roco_device_status(cache: Cache) -> int:
    flags = C.c_int32(0)
    rc = lib().roco_device_status(C.byref(cache.c), _stream(), C.byref(flags))
    if rc not in (ROCO_OK, 5):
        raise RocoError(rc, "roco_device_status")
    return int(flags.value)
