"""Thin ctypes binding of include/qsparse.h: argument marshalling only.

Every step of the synchronisation round runs in the CUDA library; PyTorch tensors supply
device memory and the stream.  Importing this module never falls back to a CPU path: if the
library cannot be loaded the import of `lib()` raises.
"""
import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

QS_OK = 0
QS_INVALID_ARG, QS_ALLOC, QS_CUDA, QS_CAPACITY, QS_NONFINITE, QS_STATE, QS_TIMEOUT = -1, -2, -3, -4, -5, -6, -7
QS_TOO_LARGE = -8
QS_STATIC_MAX_D = 1 << 20
QS_TOPK, QS_RANDK = 0, 1
QS_QSGD, QS_QSGD_SCALED, QS_SIGN_L1, QS_NONE, QS_SIGN_L2, QS_MINMAX = 0, 1, 2, 3, 4, 5
QS_ROUND_AUTO = 2**64 - 1

EXPORTS = [
    "qs_init", "qs_set_segments", "qs_set_sharding", "qs_bind", "qs_local_step", "qs_local_step_momentum", "qs_sync_round_step",
    "qs_compress_feedback", "qs_pack",
    "qs_unpack_accumulate", "qs_broadcast", "qs_sync_round", "qs_export_selection", "qs_wire_words",
    "qs_record_bits", "qs_total_k", "qs_sync_status", "qs_last_error", "qs_get_round", "qs_set_round",
    "qs_get_stats", "qs_enable_phase_timing", "qs_get_phase_timing", "qs_get_stage_trace", "qs_unpack_accumulate_static",
    "qs_gap_words", "qs_recode_gaps", "qs_decode_gaps", "qs_destroy",
]

_lib = None


def QS_OP(sparsifier, quantizer):
    return sparsifier | (quantizer << 4)


def lib():
    """Loads (building first if the sources are newer) the in-tree CUDA library."""
    global _lib
    if _lib is None:
        path = _build.build()
        if not os.path.exists(path):
            raise RuntimeError("libqsparse.so is missing: build it with paper_1906_02367_b200/build.py")
        L = C.CDLL(path)
        vp, i64, u64 = C.c_void_p, C.c_int64, C.c_uint64
        L.qs_init.argtypes = [C.POINTER(vp), C.c_int, i64, i64, C.c_int, C.c_int, u64, vp]
        L.qs_set_segments.argtypes = [vp, C.c_int, vp, vp]
        L.qs_bind.argtypes = [vp, vp, vp, vp, vp]
        L.qs_set_sharding.argtypes = [vp, C.c_int, C.c_int]
        L.qs_local_step.argtypes = [vp, vp, C.c_float, vp]
        L.qs_local_step_momentum.argtypes = [vp, vp, vp, C.c_float, C.c_float, vp]
        L.qs_sync_round_step.argtypes = [vp, vp, vp, C.c_float, C.c_float, u64, vp, vp, i64, vp]
        L.qs_compress_feedback.argtypes = [vp, u64, vp]
        L.qs_pack.argtypes = [vp, vp, i64, vp]
        L.qs_unpack_accumulate.argtypes = [vp, vp, i64, vp]
        L.qs_broadcast.argtypes = [vp, vp]
        L.qs_sync_round.argtypes = [vp, u64, vp, vp, i64, vp]
        L.qs_export_selection.argtypes = [vp, vp, vp, vp, vp, vp]
        L.qs_wire_words.argtypes = [vp]
        L.qs_wire_words.restype = i64
        L.qs_record_bits.argtypes = [vp, vp]
        L.qs_record_bits.restype = i64
        L.qs_total_k.argtypes = [vp]
        L.qs_total_k.restype = i64
        L.qs_gap_words.argtypes = [vp]
        L.qs_gap_words.restype = i64
        L.qs_recode_gaps.argtypes = [vp, vp, i64, vp, vp, i64, vp]
        L.qs_decode_gaps.argtypes = [vp, vp, i64, vp, vp, i64]
        L.qs_sync_status.argtypes = [vp]
        L.qs_last_error.argtypes = [vp]
        L.qs_last_error.restype = C.c_char_p
        L.qs_get_round.argtypes = [vp]
        L.qs_get_round.restype = u64
        L.qs_set_round.argtypes = [vp, u64]
        L.qs_get_stats.argtypes = [vp, vp, C.c_int]
        L.qs_enable_phase_timing.argtypes = [vp, C.c_int]
        L.qs_get_phase_timing.argtypes = [vp, vp, C.c_int]
        L.qs_get_stage_trace.argtypes = [vp, vp, C.c_int]
        L.qs_unpack_accumulate_static.argtypes = [C.c_int, i64, i64, C.c_int, C.c_int, vp, vp, i64, vp, vp]
        L.qs_destroy.argtypes = [vp]
        L.qs_destroy.restype = None
        _lib = L
    return _lib


class QsError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"qsparse error {code}: {text}")
        self.code = code


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _mask(mask, R):
    if mask is None:
        return None, None
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    assert m.size == R
    return m, m.ctypes.data_as(C.c_void_p)


def unpack_accumulate_static(R, d, k, s, quantizer, x, wire, mask=None, stream=None):
    """qs_unpack_accumulate_static: the master update without a context and without allocating.
    Returns the status code (0 on success) instead of raising, so that callers can test limits."""
    m, mp = _mask(mask, R)
    st = stream if stream is not None else torch.cuda.current_stream()
    return int(lib().qs_unpack_accumulate_static(int(R), int(d), int(k), int(s), int(quantizer), _ptr(x), _ptr(wire),
                                                 int(wire.shape[1]), mp, C.c_void_p(st.cuda_stream)))


class Context:
    """One qs_ctx.  Methods mirror the C calls one to one and raise QsError on a negative status."""

    def __init__(self, R, d, k, s, sparsifier=QS_TOPK, quantizer=QS_QSGD, seed=0, stream=None):
        self.R, self.d = int(R), int(d)
        self._h = C.c_void_p()
        self._stream = stream if stream is not None else torch.cuda.current_stream()
        rc = lib().qs_init(C.byref(self._h), int(R), int(d), int(k), int(s), QS_OP(sparsifier, quantizer),
                           int(seed), C.c_void_p(self._stream.cuda_stream))
        if rc != QS_OK:
            raise QsError(rc, "qs_init failed")
        self._keep = []
        self.nseg = 1
        self.R_total = self.R

    def _check(self, rc):
        if rc < 0:
            raise QsError(rc, lib().qs_last_error(self._h).decode())
        return rc

    def set_segments(self, offsets, k_seg):
        off = np.ascontiguousarray(offsets, dtype=np.int64)
        ks = np.ascontiguousarray(k_seg, dtype=np.int64)
        self._check(lib().qs_set_segments(self._h, len(ks), off.ctypes.data_as(C.c_void_p),
                                          ks.ctypes.data_as(C.c_void_p)))
        self.nseg = len(ks)

    def set_sharding(self, worker_base, R_total):
        self._check(lib().qs_set_sharding(self._h, int(worker_base), int(R_total)))
        self.R_total = int(R_total)

    def bind(self, x, xw, mem, anchors=None):
        for t in (x, xw, mem) + ((anchors,) if anchors is not None else ()):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
        assert x.numel() == self.d and xw.numel() == self.R * self.d and mem.numel() == self.R * self.d
        self._keep = [x, xw, mem, anchors]
        self._check(lib().qs_bind(self._h, _ptr(x), _ptr(xw), _ptr(mem), _ptr(anchors)))

    def local_step(self, grad, eta, mask=None):
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.is_contiguous()
        m, mp = _mask(mask, self.R)
        self._check(lib().qs_local_step(self._h, _ptr(grad), float(eta), mp))

    def local_step_momentum(self, grad, vel, eta, mu, mask=None):
        for t in (grad, vel):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
        m, mp = _mask(mask, self.R)
        self._check(lib().qs_local_step_momentum(self._h, _ptr(grad), _ptr(vel), float(eta), float(mu), mp))

    def sync_round_step(self, wire, grad, eta, vel=None, mu=0.0, rnd=QS_ROUND_AUTO, mask=None, bits_out=None):
        """The local step (with momentum when vel is given) taken inside the round."""
        for t in (grad, vel):
            assert t is None or (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous())
        m, mp = _mask(mask, self.R)
        self._check(lib().qs_sync_round_step(self._h, _ptr(grad), _ptr(vel), float(eta), float(mu), int(rnd), mp,
                                             _ptr(wire), int(wire.shape[1]), _ptr(bits_out)))

    def compress_feedback(self, rnd=QS_ROUND_AUTO, mask=None):
        m, mp = _mask(mask, self.R)
        self._check(lib().qs_compress_feedback(self._h, int(rnd), mp))

    def pack(self, wire, bits_out=None):
        assert wire.is_cuda and wire.dtype == torch.int32 and wire.is_contiguous() and wire.shape[0] == self.R
        self._check(lib().qs_pack(self._h, _ptr(wire), int(wire.shape[1]), _ptr(bits_out)))

    def unpack_accumulate(self, wire, mask=None):
        m, mp = _mask(mask, self.R_total)        # the records of the whole job
        self._check(lib().qs_unpack_accumulate(self._h, _ptr(wire), int(wire.shape[1]), mp))

    def gap_words(self):
        return int(lib().qs_gap_words(self._h))

    def recode_gaps(self, wire, packed, mask=None, bits_out=None):
        m, mp = _mask(mask, self.R)              # this context's workers; decode_gaps takes the whole job's
        self._check(lib().qs_recode_gaps(self._h, _ptr(wire), int(wire.shape[1]), mp, _ptr(packed), int(packed.shape[1]),
                                         _ptr(bits_out)))

    def decode_gaps(self, packed, wire, mask=None):
        m, mp = _mask(mask, self.R_total)
        self._check(lib().qs_decode_gaps(self._h, _ptr(packed), int(packed.shape[1]), mp, _ptr(wire), int(wire.shape[1])))

    def broadcast(self, mask=None):
        m, mp = _mask(mask, self.R)
        self._check(lib().qs_broadcast(self._h, mp))

    def sync_round(self, wire, rnd=QS_ROUND_AUTO, mask=None, bits_out=None):
        m, mp = _mask(mask, self.R)
        self._check(lib().qs_sync_round(self._h, int(rnd), mp, _ptr(wire), int(wire.shape[1]), _ptr(bits_out)))

    def export_selection(self):
        """(sel_idx R x K int64, level R x K int32, sign R x K uint8, norm, n) as device tensors."""
        K, dev = self.total_k(), self._keep[0].device
        nseg = self.nseg
        sel = torch.empty((self.R, K), dtype=torch.int64, device=dev)
        lvl = torch.empty((self.R, K), dtype=torch.int32, device=dev)
        sgn = torch.empty((self.R, K), dtype=torch.uint8, device=dev)
        nrm = torch.empty((self.R, nseg), dtype=torch.float32, device=dev)
        n = torch.empty((self.R, nseg), dtype=torch.int64, device=dev)
        self._check(lib().qs_export_selection(self._h, _ptr(sel), _ptr(lvl), _ptr(sgn), _ptr(nrm), _ptr(n)))
        return sel, lvl, sgn, nrm, n

    def wire_words(self):
        return int(lib().qs_wire_words(self._h))

    def record_bits(self, n):
        a = np.ascontiguousarray(n, dtype=np.int64)
        return int(lib().qs_record_bits(self._h, a.ctypes.data_as(C.c_void_p)))

    def total_k(self):
        return int(lib().qs_total_k(self._h))

    def sync_status(self):
        return int(lib().qs_sync_status(self._h))

    def last_error(self):
        return lib().qs_last_error(self._h).decode()

    def get_round(self):
        return int(lib().qs_get_round(self._h))

    def set_round(self, rnd):
        self._check(lib().qs_set_round(self._h, int(rnd)))

    def stats(self):
        out = np.zeros(5, dtype=np.int64)
        self._check(lib().qs_get_stats(self._h, out.ctypes.data_as(C.c_void_p), 5))
        return {"rounds": int(out[0]), "fallback_worker_rounds": int(out[1]), "candidates": int(out[2]),
                "launches": int(out[3]), "persistent_blocks": int(out[4])}

    def enable_phase_timing(self, on=True):
        self._check(lib().qs_enable_phase_timing(self._h, int(bool(on))))

    def phase_timing(self):
        out = np.zeros(3, dtype=np.float64)
        self._check(lib().qs_get_phase_timing(self._h, out.ctypes.data_as(C.c_void_p), 3))
        return {"rounds": int(out[2]), "dense_pass": float(out[0]), "rest_of_round": float(out[1])}

    def stage_trace(self):
        """Microseconds at which block 0 of the last persistent kernel reached each barrier; last = end."""
        out = np.zeros(32, dtype=np.float64)
        self._check(lib().qs_get_stage_trace(self._h, out.ctypes.data_as(C.c_void_p), 32))
        return [float(v) for v in out]

    def new_wire(self):
        return torch.zeros((self.R, self.wire_words()), dtype=torch.int32, device=self._keep[0].device)

    def destroy(self):
        if self._h:
            lib().qs_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
