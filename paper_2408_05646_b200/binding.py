"""ctypes binding of libeigenattn.so: the same calls as include/eigen_attn.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used for device memory and
streams.  There is no fallback: if the library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("EIGEN_ATTN_LIB", os.path.join(_HERE, "libeigenattn.so"))   # override: another build of the library

EA_OK = 0
EA_ERR_INVALID_ARG, EA_ERR_SHAPE, EA_ERR_CAPACITY, EA_ERR_UNSUPPORTED = -1, -2, -3, -4
EA_ERR_CUDA, EA_ERR_TIMEOUT, EA_ERR_NOT_ORTHONORMAL = -5, -6, -7
EA_BF16, EA_FP32 = 0, 1
EA_CHECK_ORTHONORMAL = 0x1
EA_ROPE_PROMPT_SCRATCH = 0x2
EA_Q_PREPROJECTED, EA_OUT_LOWRANK, EA_KV_PREPROJECTED = 0x1, 0x2, 0x4
EA_OPT_DECODE_CTAS, EA_OPT_DECODE_TILE_ROWS, EA_OPT_DECODE_STAGES, EA_OPT_PREFILL_IMPL = 1, 2, 3, 4
EA_OPT_DECODE_FUSED = 5
EA_OPT_PREFILL_PROJECT = 6
EA_OPT_TEST_WAIT_GIVES_UP = 7
EA_OPT_DECODE_MIN_COPY_BYTES = 8
EA_OPT_GQA_IMPL = 9

STATUS_NAMES = {0: "EA_OK", -1: "EA_ERR_INVALID_ARG", -2: "EA_ERR_SHAPE", -3: "EA_ERR_CAPACITY",
                -4: "EA_ERR_UNSUPPORTED", -5: "EA_ERR_CUDA", -6: "EA_ERR_TIMEOUT",
                -7: "EA_ERR_NOT_ORTHONORMAL"}


class EigenAttnError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {detail}".strip())


class ea_desc(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_heads", ctypes.c_int32), ("d_head", ctypes.c_int32),
        ("n_max", ctypes.c_int32), ("dtype", ctypes.c_int32), ("max_prefill_tokens", ctypes.c_int32),
        ("r_k", ctypes.POINTER(ctypes.c_int32)), ("r_v", ctypes.POINTER(ctypes.c_int32)),
        ("U_k", ctypes.POINTER(ctypes.c_float)), ("U_v", ctypes.POINTER(ctypes.c_float)),
        ("flags", ctypes.c_uint32),
    ]


# name -> (restype, argtypes); the list mirrors include/eigen_attn.h
_vp, _i32, _i64, _u32, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_size_t
SYMBOLS = {
    "eigen_attn_cache_bytes": (_i32, [ctypes.POINTER(ea_desc), ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "eigen_attn_create": (_i32, [ctypes.POINTER(ea_desc), _vp, _sz, _vp, _sz, _vp, ctypes.POINTER(_vp)]),
    "eigen_attn_destroy": (None, [_vp]),
    "eigen_attn_append_kv": (_i32, [_vp, _vp, _vp, _i32, _i64, _i64, _u32, _vp]),
    "eigen_attn_decode": (_i32, [_vp, _vp, _i64, _vp, _i64, _u32, _vp]),
    "eigen_attn_decode_static": (_i32, [_vp, _vp, _i64, _vp, _i64, _u32, _vp]),
    "eigen_attn_decode_step": (_i32, [_vp, _vp, _i64, _vp, _vp, _i64, _vp, _i64, _u32, _vp]),
    "eigen_attn_decode_step_host": (_i32, [_vp, _vp, _vp, _vp, _vp, _u32, _vp]),
    "eigen_attn_prefill": (_i32, [_vp, _vp, _vp, _vp, _i32, _i64, _i64, _vp, _i64, _i64, _u32, _vp]),
    "eigen_attn_get_len": (_i32, [_vp, ctypes.POINTER(_i32)]),
    "eigen_attn_set_len": (_i32, [_vp, _i32]),
    "eigen_attn_set_lens": (_i32, [_vp, ctypes.POINTER(_i32), _vp]),
    "eigen_attn_get_lens": (_i32, [_vp, ctypes.POINTER(_i32)]),
    "eigen_attn_set_page_table": (_i32, [_vp, ctypes.POINTER(_i32), _i32, _i32, _vp]),
    "eigen_attn_poll_status": (_i32, [_vp, _vp]),
    "eigen_attn_last_error": (ctypes.c_char_p, [_vp]),
    "eigen_attn_head_offsets": (_i32, [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "eigen_attn_cache_layout": (_i32, [_vp, _i32, ctypes.POINTER(_sz), ctypes.POINTER(_sz),
                                       ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "eigen_attn_set_option": (_i32, [_vp, _i32, _i64]),
    "eigen_attn_set_alibi": (_i32, [_vp, ctypes.POINTER(ctypes.c_float), _vp]),
    "eigen_attn_set_rope": (_i32, [_vp, ctypes.c_double, _i32, _vp]),
    "eigen_attn_decode_gqa": (_i32, [_vp, _vp, _i64, _i32, _vp, _i64, _vp]),
    "eigen_attn_quant_bytes": (_i32, [_vp, _i32, _i32, ctypes.POINTER(_sz)]),
    "eigen_attn_quant_attach": (_i32, [_vp, _i32, _i32, _vp, _sz, _vp]),
    "eigen_attn_quant_sync": (_i32, [_vp, _vp]),
    "eigen_attn_decode_quant": (_i32, [_vp, _vp, _i64, _vp, _i64, _u32, _vp]),
    "eigen_attn_quant_len": (_i32, [_vp, ctypes.POINTER(_i32)]),
    "eigen_attn_quant_lens": (_i32, [_vp, ctypes.POINTER(_i32)]),
    "eigen_attn_quant_layout": (_i32, [_vp, _i32] + [ctypes.POINTER(_sz)] * 5),
    "eigen_attn_launch_count": (_i32, [_vp, ctypes.POINTER(ctypes.c_uint64)]),
    "eigen_attn_set_decode_events": (_i32, [_vp, _vp, _vp]),
    "eigen_attn_version": (_i32, []),
}


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2408_05646_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    for name, (res, args) in SYMBOLS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


lib = load_library()


def device_alloc(nbytes: int, device: torch.device) -> torch.Tensor:
    """Every device buffer this module hands to the library (cache, workspace, quantised buffer, outputs it
    creates itself) comes from this function: a flat uint8 tensor whose address is a multiple of 256.  It is a
    module attribute so that a caller can substitute its own allocator, e.g. one that surrounds each buffer with
    guard regions."""
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _make_desc(batch, n_heads, d_head, n_max, dtype, r_k, r_v, U_k, U_v, max_prefill_tokens, flags):
    """Returns (desc, keepalive): ctypes arrays must outlive the call that reads them."""
    rk = (ctypes.c_int32 * n_heads)(*[int(r) for r in r_k])
    rv = (ctypes.c_int32 * n_heads)(*[int(r) for r in (r_v if r_v is not None else r_k)])
    keep = [rk, rv]
    d = ea_desc()
    d.batch, d.n_heads, d.d_head, d.n_max = batch, n_heads, d_head, n_max
    d.dtype = dtype
    d.max_prefill_tokens = max_prefill_tokens
    d.r_k = rk
    d.r_v = rv
    if U_k is not None:
        uk = np.ascontiguousarray(np.concatenate([np.asarray(u, dtype=np.float32).reshape(-1) for u in U_k]))
        uv = np.ascontiguousarray(np.concatenate([np.asarray(u, dtype=np.float32).reshape(-1) for u in U_v]))
        keep += [uk, uv]
        d.U_k = uk.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
        d.U_v = uv.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    d.flags = flags
    return d, keep


def cache_bytes(batch, n_heads, d_head, n_max, dtype, r_k, r_v=None, max_prefill_tokens=0):
    """eigen_attn_cache_bytes: (cache_bytes, workspace_bytes).  Host arithmetic only."""
    d, _keep = _make_desc(batch, n_heads, d_head, n_max, dtype, r_k, r_v, None, None, max_prefill_tokens, 0)
    cb, wb = _sz(0), _sz(0)
    st = lib.eigen_attn_cache_bytes(ctypes.byref(d), ctypes.byref(cb), ctypes.byref(wb))
    if st != EA_OK:
        raise EigenAttnError(st, "eigen_attn_cache_bytes")
    return cb.value, wb.value


class EigenAttnLayer:
    """One decoder layer's rank-r KV cache and the library calls on it (eigen_attn_t)."""

    def __init__(self, batch: int, n_heads: int, d_head: int, n_max: int, dtype: torch.dtype,
                 U_k: Sequence[np.ndarray], U_v: Sequence[np.ndarray], max_prefill_tokens: int = 0,
                 device: str | torch.device = "cuda:0", check_orthonormal: bool = False,
                 stream: Optional[torch.cuda.Stream] = None, rope_prompt_scratch: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("EigenAttnLayer needs a CUDA device; there is no CPU fallback")
        self.B, self.H, self.d_head, self.n_max = batch, n_heads, d_head, n_max
        self.torch_dtype = dtype
        self.ea_dtype = {torch.bfloat16: EA_BF16, torch.float32: EA_FP32}[dtype]
        self.device = torch.device(device)
        self.r_k = [int(u.shape[1]) for u in U_k]
        self.r_v = [int(u.shape[1]) for u in U_v]
        for u in list(U_k) + list(U_v):
            assert u.shape[0] == d_head
        desc, keep = _make_desc(batch, n_heads, d_head, n_max, self.ea_dtype, self.r_k, self.r_v, U_k, U_v,
                                max_prefill_tokens, (EA_CHECK_ORTHONORMAL if check_orthonormal else 0) |
                                (EA_ROPE_PROMPT_SCRATCH if rope_prompt_scratch else 0))
        cb, wb = _sz(0), _sz(0)
        st = lib.eigen_attn_cache_bytes(ctypes.byref(desc), ctypes.byref(cb), ctypes.byref(wb))
        if st != EA_OK:
            raise EigenAttnError(st, "eigen_attn_cache_bytes")
        with torch.cuda.device(self.device):
            self.cache = device_alloc(cb.value, self.device)
            self.workspace = device_alloc(wb.value, self.device)
            handle = _vp(0)
            st = lib.eigen_attn_create(ctypes.byref(desc), self.cache.data_ptr(), cb.value,
                                       self.workspace.data_ptr(), wb.value, _stream_ptr(stream),
                                       ctypes.byref(handle))
        del keep
        if st != EA_OK:
            raise EigenAttnError(st, "eigen_attn_create")
        self.handle = handle
        offs_k = (ctypes.c_int32 * (n_heads + 1))()
        offs_v = (ctypes.c_int32 * (n_heads + 1))()
        self._check(lib.eigen_attn_head_offsets(self.handle, offs_k, offs_v), "eigen_attn_head_offsets")
        self.offs_k, self.offs_v = list(offs_k), list(offs_v)

    # -- plumbing
    def _new_out(self, *shape) -> torch.Tensor:
        es = 2 if self.torch_dtype == torch.bfloat16 else 4
        n = 1
        for d in shape:
            n *= int(d)
        return device_alloc(n * es, self.device).view(self.torch_dtype).view(*shape)

    def _check(self, st: int, where: str) -> None:
        if st != EA_OK:
            raise EigenAttnError(st, where, lib.eigen_attn_last_error(self.handle).decode())

    def close(self) -> None:
        if getattr(self, "handle", None):
            lib.eigen_attn_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _tok(self, x: torch.Tensor, T: Optional[int] = None):
        """Checks a [B][T][H][d_head] tensor and returns (ptr, T, stride_b, stride_t)."""
        assert x.is_cuda and x.dtype == self.torch_dtype and x.dim() == 4
        assert x.shape[0] == self.B and x.shape[2] == self.H and x.shape[3] == self.d_head
        assert x.stride(3) == 1 and x.stride(2) == self.d_head
        if T is not None:
            assert x.shape[1] == T
        return x.data_ptr(), x.shape[1], x.stride(0), x.stride(1)

    # -- the calls of include/eigen_attn.h
    def append_kv(self, k: torch.Tensor, v: torch.Tensor, preprojected: bool = False, stream=None) -> None:
        if preprojected:
            assert k.is_contiguous() and v.is_contiguous() and k.dtype == self.torch_dtype
            assert k.shape == (self.B, k.shape[1], self.offs_k[-1]) and v.shape == (self.B, k.shape[1], self.offs_v[-1])
            T = k.shape[1]
            st = lib.eigen_attn_append_kv(self.handle, k.data_ptr(), v.data_ptr(), T, k.stride(0), k.stride(1),
                                          EA_KV_PREPROJECTED, _stream_ptr(stream))
            self._check(st, "eigen_attn_append_kv")
            return
        pk, T, sb, stt = self._tok(k)
        pv, _, sb2, st2 = self._tok(v, T)
        assert (sb, stt) == (sb2, st2)
        self._check(lib.eigen_attn_append_kv(self.handle, pk, pv, T, sb, stt, 0, _stream_ptr(stream)),
                    "eigen_attn_append_kv")

    def decode(self, q: torch.Tensor, out: Optional[torch.Tensor] = None, q_preprojected: bool = False,
               out_lowrank: bool = False, stream=None, _fn=None, _name="eigen_attn_decode") -> torch.Tensor:
        flags = 0
        if q_preprojected:
            assert q.is_contiguous() and q.shape == (self.B, 1, self.offs_k[-1]) and q.dtype == self.torch_dtype
            flags |= EA_Q_PREPROJECTED
            pq, sbq = q.data_ptr(), self.offs_k[-1]
        else:
            pq, _, sbq, _ = self._tok(q, 1)
        if out_lowrank:
            flags |= EA_OUT_LOWRANK
            if out is None:
                out = self._new_out(self.B, 1, self.offs_v[-1])
            assert out.is_contiguous() and out.dtype == self.torch_dtype
            sbo = self.offs_v[-1]
        else:
            if out is None:
                out = self._new_out(self.B, 1, self.H, self.d_head)
            _, _, sbo, _ = self._tok(out, 1)
        fn = _fn if _fn is not None else lib.eigen_attn_decode
        self._check(fn(self.handle, pq, sbq, out.data_ptr(), sbo, flags, _stream_ptr(stream)), _name)
        return out

    # -- quantised copy of the cache (4-bit codes, one half-precision scale per group)
    def quant_bytes(self, bits: int, group: int) -> int:
        n = _sz(0)
        self._check(lib.eigen_attn_quant_bytes(self.handle, int(bits), int(group), ctypes.byref(n)), "eigen_attn_quant_bytes")
        return n.value

    def quant_attach(self, bits: int, group: int, stream=None) -> torch.Tensor:
        """Allocates the quantised buffer (a torch byte tensor kept on the layer) and attaches it."""
        nbytes = self.quant_bytes(bits, group)
        self.qcache = device_alloc(nbytes, self.device).zero_()
        self.q_group = int(group)
        self._check(lib.eigen_attn_quant_attach(self.handle, int(bits), int(group), self.qcache.data_ptr(), nbytes,
                                                _stream_ptr(stream)), "eigen_attn_quant_attach")
        return self.qcache

    def quant_detach(self, stream=None) -> None:
        """Detaches the quantised buffer (eigen_attn_quant_attach with NULL) and drops the tensor."""
        self._check(lib.eigen_attn_quant_attach(self.handle, 0, 0, None, 0, _stream_ptr(stream)), "eigen_attn_quant_attach")
        self.qcache = None

    def quant_sync(self, stream=None) -> None:
        self._check(lib.eigen_attn_quant_sync(self.handle, _stream_ptr(stream)), "eigen_attn_quant_sync")

    @property
    def quant_len(self) -> int:
        n = ctypes.c_int32(0)
        self._check(lib.eigen_attn_quant_len(self.handle, ctypes.byref(n)), "eigen_attn_quant_len")
        return n.value

    def quant_lens(self):
        arr = (ctypes.c_int32 * self.B)()
        self._check(lib.eigen_attn_quant_lens(self.handle, arr), "eigen_attn_quant_lens")
        return list(arr)

    def decode_quant(self, q: torch.Tensor, out: Optional[torch.Tensor] = None, q_preprojected: bool = False,
                     out_lowrank: bool = False, stream=None) -> torch.Tensor:
        return self.decode(q, out, q_preprojected, out_lowrank, stream, _fn=lib.eigen_attn_decode_quant,
                           _name="eigen_attn_decode_quant")

    def quant_layout(self, head: int):
        """(slab offset, block bytes, key-scale offset, value-code offset, value-scale offset) of a head."""
        v = [_sz(0) for _ in range(5)]
        self._check(lib.eigen_attn_quant_layout(self.handle, int(head), *[ctypes.byref(x) for x in v]),
                    "eigen_attn_quant_layout")
        return tuple(x.value for x in v)

    def quant_blocks(self, head: int) -> torch.Tensor:
        """View of head `head`'s slab [B][n_max // group][block_bytes] of the quantised buffer (for inspection)."""
        slab, bb, _, _, _ = self.quant_layout(head)
        nb = self.n_max // self.q_group
        return self.qcache[slab:slab + self.B * nb * bb].view(self.B, nb, bb)

    def decode_static(self, q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """eigen_attn_decode_static: decode with the partials in the library's built-in scratch array
        (for callers that cannot hand the call any scratch memory).  Calls that could overlap on the
        GPU share that array and must be serialised."""
        pq, _, sbq, _ = self._tok(q, 1)
        if out is None:
            out = self._new_out(self.B, 1, self.H, self.d_head)
        _, _, sbo, _ = self._tok(out, 1)
        self._check(lib.eigen_attn_decode_static(self.handle, pq, sbq, out.data_ptr(), sbo, 0,
                                                 _stream_ptr(stream)), "eigen_attn_decode_static")
        return out

    def _packed(self, x: torch.Tensor, T: int, width: int) -> int:
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.torch_dtype and x.shape == (self.B, T, width)
        return x.data_ptr()

    def decode_step(self, q, k, v, out: Optional[torch.Tensor] = None, q_preprojected: bool = False,
                    kv_preprojected: bool = False, out_lowrank: bool = False, stream=None) -> torch.Tensor:
        flags = 0
        if q_preprojected:
            flags |= EA_Q_PREPROJECTED
            pq, sbq = self._packed(q, 1, self.offs_k[-1]), self.offs_k[-1]
        else:
            pq, _, sbq, _ = self._tok(q, 1)
        if kv_preprojected:
            flags |= EA_KV_PREPROJECTED
            pk, pv, sbk = self._packed(k, 1, self.offs_k[-1]), self._packed(v, 1, self.offs_v[-1]), 0
        else:
            pk, _, sbk, _ = self._tok(k, 1)
            pv, _, sbv, _ = self._tok(v, 1)
            if sbk != sbv:
                k, v = k.contiguous(), v.contiguous()
                pk, _, sbk, _ = self._tok(k, 1)
                pv, _, sbv, _ = self._tok(v, 1)
        if out_lowrank:
            flags |= EA_OUT_LOWRANK
            if out is None:
                out = self._new_out(self.B, 1, self.offs_v[-1])
            po, sbo = self._packed(out, 1, self.offs_v[-1]), self.offs_v[-1]
        else:
            if out is None:
                out = self._new_out(self.B, 1, self.H, self.d_head)
            po, _, sbo, _ = self._tok(out, 1)
        self._check(lib.eigen_attn_decode_step(self.handle, pq, sbq, pk, pv, sbk, po, sbo, flags, _stream_ptr(stream)),
                    "eigen_attn_decode_step")
        return out

    def decode_step_host(self, h_q, h_k, h_v, h_out, stream=None) -> torch.Tensor:
        """Host tensors (contiguous, ideally pinned) in, host tensor out; synchronises the stream."""
        for x in (h_q, h_k, h_v, h_out):
            assert not x.is_cuda and x.is_contiguous() and x.dtype == self.torch_dtype
            assert x.numel() == self.B * self.H * self.d_head
        self._check(lib.eigen_attn_decode_step_host(self.handle, h_q.data_ptr(), h_k.data_ptr(), h_v.data_ptr(),
                                                    h_out.data_ptr(), 0, _stream_ptr(stream)),
                    "eigen_attn_decode_step_host")
        return h_out

    def prefill(self, q, k, v, out: Optional[torch.Tensor] = None, out_lowrank: bool = False,
                q_preprojected: bool = False, kv_preprojected: bool = False, stream=None):
        T = q.shape[1]
        flags = 0
        strides = []
        if q_preprojected:
            flags |= EA_Q_PREPROJECTED
            pq = self._packed(q, T, self.offs_k[-1])
        else:
            pq, _, sb, stt = self._tok(q, T)
            strides.append((sb, stt))
        if kv_preprojected:
            flags |= EA_KV_PREPROJECTED
            pk, pv = self._packed(k, T, self.offs_k[-1]), self._packed(v, T, self.offs_v[-1])
        else:
            pk, _, sbk, stk = self._tok(k, T)
            pv, _, sbv, stv = self._tok(v, T)
            strides += [(sbk, stk), (sbv, stv)]
        assert len(set(strides)) <= 1                    # the d_head-wide tensors share their strides
        sb, stt = strides[0] if strides else (0, 0)
        if out_lowrank:
            flags |= EA_OUT_LOWRANK
            if out is None:
                out = self._new_out(self.B, T, self.offs_v[-1])
            assert out.is_contiguous()
            po, sbo, sto = out.data_ptr(), T * self.offs_v[-1], self.offs_v[-1]
        else:
            if out is None:
                out = self._new_out(self.B, T, self.H, self.d_head)
            po, _, sbo, sto = self._tok(out, T)
        self._check(lib.eigen_attn_prefill(self.handle, pq, pk, pv, T, sb, stt, po, sbo, sto, flags, _stream_ptr(stream)),
                    "eigen_attn_prefill")
        return out

    @property
    def len(self) -> int:
        n = ctypes.c_int32(0)
        self._check(lib.eigen_attn_get_len(self.handle, ctypes.byref(n)), "eigen_attn_get_len")
        return n.value

    def set_len(self, n: int) -> None:
        self._check(lib.eigen_attn_set_len(self.handle, int(n)), "eigen_attn_set_len")

    def set_lens(self, lens, stream=None) -> None:
        """Per-sequence lengths of a batch whose sequences differ in length (host integers, one per sequence)."""
        arr = (ctypes.c_int32 * self.B)(*[int(x) for x in lens])
        self._check(lib.eigen_attn_set_lens(self.handle, arr, _stream_ptr(stream)), "eigen_attn_set_lens")

    def lens(self):
        arr = (ctypes.c_int32 * self.B)()
        self._check(lib.eigen_attn_get_lens(self.handle, arr), "eigen_attn_get_lens")
        return list(arr)

    def set_page_table(self, table, page_rows: int = 128, stream=None) -> None:
        """table: [batch][pages_per_seq] physical page of every logical page (-1 = not mapped); None = contiguous."""
        if table is None:
            self._check(lib.eigen_attn_set_page_table(self.handle, None, 0, 0, _stream_ptr(stream)), "eigen_attn_set_page_table")
            return
        width = len(table[0])
        assert len(table) == self.B and all(len(r) == width for r in table)
        arr = (ctypes.c_int32 * (self.B * width))(*[int(x) for r in table for x in r])
        self._check(lib.eigen_attn_set_page_table(self.handle, arr, width, int(page_rows), _stream_ptr(stream)),
                    "eigen_attn_set_page_table")

    def poll_status(self, stream=None) -> None:
        self._check(lib.eigen_attn_poll_status(self.handle, _stream_ptr(stream)), "eigen_attn_poll_status")

    def set_alibi(self, slopes, stream=None) -> None:
        """Per-head ALiBi slopes (host floats, one per head); None switches the bias off."""
        if slopes is None:
            arr = None
        else:
            assert len(slopes) == self.H
            arr = (ctypes.c_float * self.H)(*[float(x) for x in slopes])
        self._check(lib.eigen_attn_set_alibi(self.handle, arr, _stream_ptr(stream)), "eigen_attn_set_alibi")

    def decode_gqa(self, q: torch.Tensor, group: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """eigen_attn_decode_gqa: q [B][1][H * group][d_head]; the layer's heads are the K/V heads."""
        assert q.shape == (self.B, 1, self.H * group, self.d_head) and q.dtype == self.torch_dtype
        assert q.stride(3) == 1 and q.stride(2) == self.d_head
        if out is None:
            out = self._new_out(self.B, 1, self.H * group, self.d_head)
        assert out.stride(3) == 1 and out.stride(2) == self.d_head
        self._check(lib.eigen_attn_decode_gqa(self.handle, q.data_ptr(), q.stride(0), int(group), out.data_ptr(),
                                              out.stride(0), _stream_ptr(stream)), "eigen_attn_decode_gqa")
        return out

    def set_rope(self, base: float, interleaved: bool = False, stream=None) -> None:
        """Rotary position embedding for decode (Section 4.3); base 0 switches it off."""
        self._check(lib.eigen_attn_set_rope(self.handle, float(base), int(bool(interleaved)), _stream_ptr(stream)),
                    "eigen_attn_set_rope")

    def set_option(self, option: int, value: int) -> None:
        self._check(lib.eigen_attn_set_option(self.handle, option, int(value)), "eigen_attn_set_option")

    def launch_count(self) -> int:
        n = ctypes.c_uint64(0)
        self._check(lib.eigen_attn_launch_count(self.handle, ctypes.byref(n)), "eigen_attn_launch_count")
        return n.value

    def set_decode_events(self, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
        a = start.cuda_event if start is not None else None
        b = stop.cuda_event if stop is not None else None
        self._check(lib.eigen_attn_set_decode_events(self.handle, a, b), "eigen_attn_set_decode_events")

    def cache_layout(self, head: int):
        ko, vo, rk, rv = _sz(0), _sz(0), ctypes.c_int32(0), ctypes.c_int32(0)
        self._check(lib.eigen_attn_cache_layout(self.handle, head, ctypes.byref(ko), ctypes.byref(vo),
                                                ctypes.byref(rk), ctypes.byref(rv)), "eigen_attn_cache_layout")
        return ko.value, vo.value, rk.value, rv.value

    def cache_rows(self, head: int, which: str = "k") -> torch.Tensor:
        """View of head `head`'s slab [B][n_max][rp] inside the cache buffer (for inspection)."""
        ko, vo, rk, rv = self.cache_layout(head)
        off, rp = (ko, rk) if which == "k" else (vo, rv)
        es = 2 if self.torch_dtype == torch.bfloat16 else 4
        nbytes = self.B * self.n_max * rp * es
        return self.cache[off:off + nbytes].view(self.torch_dtype).view(self.B, self.n_max, rp)
