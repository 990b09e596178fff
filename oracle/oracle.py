"""ctypes access to the CPU oracle (oracle/qs_oracle.cpp).

Test infrastructure only: imported by the tests, the smoke check and the CPU
baseline leg of the benchmark.  Nothing here touches the CUDA library.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

TOPK, RANDK = 0, 1
QSGD, QSGD_SCALED, SIGN_L1, NONE, SIGN_L2, MINMAX = 0, 1, 2, 3, 4, 5
SORT, NTH = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.qso_philox_word.restype = C.c_uint32
        _lib.qso_philox_word.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint32]
        _lib.qso_norm_l2.restype = C.c_float
        _lib.qso_norm_l1.restype = C.c_float
        _lib.qso_qsgd_level.restype = C.c_int
        _lib.qso_qsgd_level.argtypes = [C.c_float, C.c_float, C.c_int, C.c_uint32]
        _lib.qso_minmax_level.restype = C.c_int
        _lib.qso_minmax_level.argtypes = [C.c_float, C.c_float, C.c_float, C.c_int, C.c_uint32]
        _lib.qso_value_minmax.restype = C.c_float
        _lib.qso_value_minmax.argtypes = [C.c_float, C.c_float, C.c_int, C.c_int]
        _lib.qso_beta_qsgd.restype = C.c_double
        _lib.qso_beta_qsgd.argtypes = [C.c_int64, C.c_int]
        _lib.qso_wire_words.restype = C.c_int64
        _lib.qso_gap_words.restype = C.c_int64
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _f32(a):
    assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]
    return _p(a, C.c_float)


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().qso_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def philox_word(seed, rnd, worker, element, stream):
    return int(lib().qso_philox_word(seed, rnd, worker, element, stream))


def norm_l2(v):
    v = np.ascontiguousarray(v, dtype=np.float32)
    return np.float32(lib().qso_norm_l2(_f32(v), C.c_int64(v.size)))


def norm_l1(v):
    v = np.ascontiguousarray(v, dtype=np.float32)
    return np.float32(lib().qso_norm_l1(_f32(v), C.c_int64(v.size)))


def select_topk(u, k, mode=SORT):
    u = np.ascontiguousarray(u, dtype=np.float32)
    out = np.zeros(k, dtype=np.int64)
    lib().qso_select_topk(_f32(u), C.c_int64(u.size), C.c_int64(k), C.c_int(mode), _p(out, C.c_int64))
    return out


def select_randk(seed, rnd, worker, lo, n, k, mode=SORT):
    out = np.zeros(k, dtype=np.int64)
    lib().qso_select_randk(C.c_uint64(seed), C.c_uint64(rnd), C.c_uint32(worker), C.c_int64(lo),
                           C.c_int64(n), C.c_int64(k), C.c_int(mode), _p(out, C.c_int64))
    return out


def qsgd_level(u, N, s, w):
    return int(lib().qso_qsgd_level(C.c_float(u), C.c_float(N), s, w))


def minmax_level(v, lo, hi, s, w):
    return int(lib().qso_minmax_level(C.c_float(v), C.c_float(lo), C.c_float(hi), s, w))


def value_minmax(lo, hi, s, level):
    return float(lib().qso_value_minmax(C.c_float(lo), C.c_float(hi), s, level))


def beta_qsgd(k, s):
    return float(lib().qso_beta_qsgd(k, s))


class Plan:
    """Operator configuration: R workers, d coordinates, segments with their k."""

    def __init__(self, R, d, k=None, s=16, sparsifier=TOPK, quantizer=QSGD, seed=0,
                 offsets=None, kseg=None):
        self.R, self.d, self.s = int(R), int(d), int(s)
        self.sparsifier, self.quantizer, self.seed = sparsifier, quantizer, int(seed)
        if offsets is None:
            offsets, kseg = [0, d], [k]
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        self.kseg = np.ascontiguousarray(kseg, dtype=np.int64)
        self.nseg = len(self.kseg)
        self.K = int(self.kseg.sum())

    def _head(self):
        return (C.c_int(self.R), C.c_int64(self.d), C.c_int(self.nseg), _p(self.offsets, C.c_int64),
                _p(self.kseg, C.c_int64), C.c_int(self.s))

    def wire_words(self):
        return int(lib().qso_wire_words(*self._head(), C.c_int(self.quantizer)))


def _mask(mask):
    return None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)


def local_step(plan, xw, grad, eta, mask=None):
    m = _mask(mask)
    lib().qso_local_step(C.c_int(plan.R), C.c_int64(plan.d), _f32(xw), _f32(grad), C.c_float(eta),
                         _p(m, C.c_uint8))


def local_step_momentum(plan, xw, vel, grad, eta, mu, mask=None):
    m = _mask(mask)
    lib().qso_local_step_momentum(C.c_int(plan.R), C.c_int64(plan.d), _f32(xw), _f32(vel), _f32(grad),
                                  C.c_float(eta), C.c_float(mu), _p(m, C.c_uint8))


def compress_feedback(plan, rnd, x, xw, mem, anchors=None, mask=None, mode=SORT, nthreads=1,
                      details=False):
    """Worker half.  Returns dict(wire, bits[, sel, level, sign, norm, n])."""
    stride = plan.wire_words()
    wire = np.zeros((plan.R, stride), dtype=np.uint32)
    bits = np.zeros(plan.R, dtype=np.int64)
    m = _mask(mask)
    out = {"wire": wire, "bits": bits, "stride": stride}
    sel = lvl = sgn = nrm = nn = None
    if details:
        sel = np.full((plan.R, plan.K), -1, dtype=np.int64)
        lvl = np.zeros((plan.R, plan.K), dtype=np.int32)
        sgn = np.zeros((plan.R, plan.K), dtype=np.uint8)
        nrm = np.zeros((plan.R, plan.nseg), dtype=np.float32)
        nn = np.zeros((plan.R, plan.nseg), dtype=np.int64)
        out.update(sel=sel, level=lvl, sign=sgn, norm=nrm, n=nn)
    rc = lib().qso_compress_feedback(
        *plan._head(), C.c_int(plan.sparsifier), C.c_int(plan.quantizer), C.c_uint64(plan.seed),
        C.c_uint64(rnd), _f32(x), _f32(xw), _f32(mem), None if anchors is None else _f32(anchors),
        _p(m, C.c_uint8), _p(wire, C.c_uint32), C.c_int64(stride), _p(bits, C.c_int64),
        C.c_int(mode), C.c_int(nthreads), _p(sel, C.c_int64), _p(lvl, C.c_int32),
        _p(sgn, C.c_uint8), _p(nrm, C.c_float), _p(nn, C.c_int64))
    out["rc"] = rc
    return out


def compress_worker(plan, rnd, worker, anchor, xw_r, mem_r, mode=NTH):
    """Worker half for the single worker `worker` on its own rows (mem_r updated in place)."""
    stride = plan.wire_words()
    wire = np.zeros(stride, dtype=np.uint32)
    bits = np.zeros(1, dtype=np.int64)
    rc = lib().qso_compress_worker(
        C.c_int64(plan.d), C.c_int(plan.nseg), _p(plan.offsets, C.c_int64), _p(plan.kseg, C.c_int64),
        C.c_int(plan.s), C.c_int(plan.sparsifier), C.c_int(plan.quantizer), C.c_uint64(plan.seed), C.c_uint64(rnd),
        C.c_int(worker), _f32(anchor), _f32(xw_r), _f32(mem_r), _p(wire, C.c_uint32), C.c_int64(stride),
        _p(bits, C.c_int64), C.c_int(mode))
    return {"rc": rc, "wire": wire, "bits": int(bits[0])}


def unpack_accumulate(plan, x, wire, mask=None):
    m = _mask(mask)
    wire = np.ascontiguousarray(wire, dtype=np.uint32)
    return lib().qso_unpack_accumulate(*plan._head(), C.c_int(plan.quantizer), _f32(x),
                                       _p(wire, C.c_uint32), C.c_int64(wire.shape[1]),
                                       _p(m, C.c_uint8))


def gap_words(plan):
    return int(lib().qso_gap_words(*plan._head(), C.c_int(plan.quantizer)))


def recode_gaps(plan, wire, mask=None):
    """Plain records -> gap-coded records (first index + gaps in fields of the widest gap's length)."""
    m = _mask(mask)
    wire = np.ascontiguousarray(wire, dtype=np.uint32)
    stride = gap_words(plan)
    out = np.zeros((plan.R, stride), dtype=np.uint32)
    bits = np.zeros(plan.R, dtype=np.int64)
    rc = lib().qso_recode_gaps(*plan._head(), C.c_int(plan.quantizer), _p(wire, C.c_uint32), C.c_int64(wire.shape[1]),
                               _p(m, C.c_uint8), _p(out, C.c_uint32), C.c_int64(stride), _p(bits, C.c_int64))
    return {"rc": rc, "packed": out, "bits": bits, "stride": stride}


def decode_gaps(plan, packed, mask=None):
    m = _mask(mask)
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    stride = plan.wire_words()
    wire = np.zeros((plan.R, stride), dtype=np.uint32)
    rc = lib().qso_decode_gaps(*plan._head(), C.c_int(plan.quantizer), _p(packed, C.c_uint32), C.c_int64(packed.shape[1]),
                               _p(m, C.c_uint8), _p(wire, C.c_uint32), C.c_int64(stride))
    return {"rc": rc, "wire": wire}


def broadcast(plan, x, xw, anchors=None, mask=None):
    m = _mask(mask)
    lib().qso_broadcast(C.c_int(plan.R), C.c_int64(plan.d), _f32(x), _f32(xw),
                        None if anchors is None else _f32(anchors), _p(m, C.c_uint8))


def sync_round(plan, rnd, x, xw, mem, anchors=None, mask=None, mode=SORT, nthreads=1):
    """Whole round in place on x, xw, mem (and anchors).  Returns dict(rc, wire, bits)."""
    stride = plan.wire_words()
    wire = np.zeros((plan.R, stride), dtype=np.uint32)
    bits = np.zeros(plan.R, dtype=np.int64)
    m = _mask(mask)
    rc = lib().qso_sync_round(
        *plan._head(), C.c_int(plan.sparsifier), C.c_int(plan.quantizer), C.c_uint64(plan.seed),
        C.c_uint64(rnd), _f32(x), _f32(xw), _f32(mem), None if anchors is None else _f32(anchors),
        _p(m, C.c_uint8), _p(wire, C.c_uint32), C.c_int64(stride), _p(bits, C.c_int64),
        C.c_int(mode), C.c_int(nthreads))
    return {"rc": rc, "wire": wire, "bits": bits, "stride": stride}
