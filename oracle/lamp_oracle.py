"""ctypes front end of the plain-C oracle in ``lamp_oracle.c``.

The C file is compiled on first use with gcc (``-ffp-contract=off`` so that only the
fused operations the source writes out are fused, ``-mfma`` so that ``fmaf`` is the
hardware instruction and not a double-precision emulation).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lamp_oracle.c")
_SO = os.path.join(_HERE, "liblamp_oracle.so")

FORCE_16BIT, FORCE_8BIT, NO_STAGE1 = 1, 2, 4
SR_E4M3 = 64          # stochastic rounding in the 8-bit accumulation (Sec. 3.3), counter-based generator
H16_SEQ = 32          # 16-bit logits by per-step e4m11 accumulation (Sec. 4.1 recursion) instead of one rounding
COMPACT_BRANCH = 16   # Sec. 3.3 'Register layout': whole tile to 16 bits once two sub-blocks are marked


class Params(C.Structure):
    _fields_ = [("batch", C.c_int32), ("heads_q", C.c_int32), ("heads_kv", C.c_int32),
                ("seqlen", C.c_int32), ("head_dim", C.c_int32), ("causal", C.c_int32),
                ("window", C.c_int32), ("scale", C.c_float), ("tau", C.c_float),
                ("delta", C.c_float), ("flags", C.c_uint32), ("sr_seed", C.c_uint32),
                ("group_rows", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("subblocks_active", C.c_uint64), ("stage1_flagged", C.c_uint64),
                ("stage2_flagged", C.c_uint64), ("hist_flagged_per_tile", C.c_uint64 * 5),
                ("sat_e4m3", C.c_uint64), ("sat_e4m11", C.c_uint64),
                ("exp16_gt1", C.c_uint64), ("big_rowsum", C.c_uint64)]

    def as_dict(self):
        d = {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "hist_flagged_per_tile"}
        d["hist_flagged_per_tile"] = [int(x) for x in self.hist_flagged_per_tile]
        return d


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-mfma", "-fopenmp", "-fPIC",
             "-shared", "-Wall", "-Wextra", _SRC, "-o", _SO, "-lm"])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        f32, f64, u8, u32 = C.c_float, C.c_double, C.c_uint8, C.c_uint32
        L.lamp_oracle_rne_e4m3.restype = f32; L.lamp_oracle_rne_e4m3.argtypes = [f32]
        L.lamp_oracle_rne_e4m11.restype = f32; L.lamp_oracle_rne_e4m11.argtypes = [f64]
        L.lamp_oracle_trunc_e4m3.restype = f32; L.lamp_oracle_trunc_e4m3.argtypes = [f32]
        L.lamp_oracle_enc_e4m3.restype = u8; L.lamp_oracle_enc_e4m3.argtypes = [f32]
        L.lamp_oracle_dec_e4m3.restype = f32; L.lamp_oracle_dec_e4m3.argtypes = [u8]
        L.lamp_oracle_enc_ue5m3.restype = u8; L.lamp_oracle_enc_ue5m3.argtypes = [f32]
        L.lamp_oracle_dec_ue5m3.restype = f32; L.lamp_oracle_dec_ue5m3.argtypes = [u8]
        L.lamp_oracle_dec_exp8.restype = f64; L.lamp_oracle_dec_exp8.argtypes = [u8]
        L.lamp_oracle_lut8.restype = u8; L.lamp_oracle_lut8.argtypes = [u8]
        L.lamp_oracle_exp16.restype = f32; L.lamp_oracle_exp16.argtypes = [f32]
        L.lamp_oracle_stage2.restype = u32
        L.lamp_oracle_stage2.argtypes = [C.c_void_p, C.c_void_p, f32, u32]
        L.lamp_oracle_sr_e4m3.restype = f32
        L.lamp_oracle_sr_e4m3.argtypes = [f32, C.c_uint32]
        L.lamp_oracle_sr_bits.restype = C.c_uint32
        L.lamp_oracle_sr_bits.argtypes = [C.c_uint32] * 5
        L.lamp_oracle_chain16.restype = f32
        L.lamp_oracle_chain16.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.lamp_oracle_chain8.restype = f32
        L.lamp_oracle_chain8.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.lamp_oracle_exp16_array.restype = None
        L.lamp_oracle_exp16_array.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        L.lamp_oracle_rne_e4m3_array.restype = None
        L.lamp_oracle_rne_e4m3_array.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.lamp_oracle_units.restype = C.c_int
        L.lamp_oracle_units.argtypes = [C.c_void_p] * 3 + [C.POINTER(Params), C.c_int64] + [C.c_void_p] * 7 + [C.POINTER(Stats)]
        _lib = L
    return _lib


def rne_e4m3_array(x: np.ndarray) -> np.ndarray:
    """The oracle's e4m3 rounding, element by element, on a float32 array."""
    x = np.ascontiguousarray(x, np.float32)
    out = np.empty_like(x)
    lib().lamp_oracle_rne_e4m3_array(x.ctypes.data_as(C.c_void_p), out.ctypes.data_as(C.c_void_p), x.size)
    return out


def exp16_array(x: np.ndarray) -> np.ndarray:
    """The oracle's 16-bit exponential, element by element, on a float32 array."""
    x = np.ascontiguousarray(x, np.float32)
    out = np.empty_like(x)
    lib().lamp_oracle_exp16_array(x.ctypes.data_as(C.c_void_p), out.ctypes.data_as(C.c_void_p), x.size)
    return out


@dataclass
class OracleResult:
    units: np.ndarray        # [n, 3] (b, h, g)
    out: np.ndarray          # [n, 32, D] fp32
    lse: np.ndarray          # [n, 32] fp32
    flags: np.ndarray        # [n, N/64] u8
    checks: np.ndarray | None  # [n, N/64, 2] u64
    y8: np.ndarray | None    # [n, 32, N] u8
    e8: np.ndarray | None    # [n, 32, N] u8
    stats: dict


def _bits(x) -> np.ndarray:
    """bf16 tensor (torch) or uint16 array -> contiguous uint16 numpy array."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return np.ascontiguousarray(x.contiguous().view(torch.int16).numpy().view(np.uint16))


def run_units(q, k, v, units, *, causal=True, window=0, scale=None, tau=0.5, delta=2.0 ** -8,
              flags=0, sr_seed=0, group_rows=0, dumps=False, checksums=True) -> OracleResult:
    """Run the oracle on the listed (b, h, g) units.  q: [B, Hq, N, D], k/v: [B, Hkv, N, D]."""
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    B, Hq, N, D = qb.shape
    Hkv = kb.shape[1]
    if scale is None:
        scale = np.float32(1.0 / np.sqrt(float(D)))
    units = np.ascontiguousarray(np.asarray(units, dtype=np.int32).reshape(-1, 3))
    n = units.shape[0]
    p = Params(B, Hq, Hkv, N, D, int(causal), int(window), float(scale), float(tau), float(delta), int(flags), int(sr_seed), int(group_rows))
    rows = 64 if int(group_rows) > 32 else 32          # rows per unit in the outputs
    out = np.zeros((n, rows, D), np.float32)
    lse = np.zeros((n, rows), np.float32)
    fl = np.zeros((n, (N + 63) // 64), np.uint8)
    ck = np.zeros((n, (N + 63) // 64, 2), np.uint64) if checksums else None
    y8 = np.zeros((n, rows, N), np.uint8) if dumps else None
    e8 = np.zeros((n, rows, N), np.uint8) if dumps else None
    st = Stats()
    ptr = lambda a: a.ctypes.data_as(C.c_void_p) if a is not None else None
    rc = lib().lamp_oracle_units(ptr(qb), ptr(kb), ptr(vb), C.byref(p), n, ptr(units), ptr(out),
                                 ptr(lse), ptr(fl), ptr(ck), ptr(y8), ptr(e8), C.byref(st))
    if rc != 0:
        raise ValueError("oracle: unsupported shape or parameters")
    return OracleResult(units, out, lse, fl, ck, y8, e8, st.as_dict())


def all_units(B, Hq, N, group_rows=32):
    g = np.stack(np.meshgrid(np.arange(B), np.arange(Hq), np.arange((N + group_rows - 1) // group_rows),
                             indexing="ij"), -1)
    return g.reshape(-1, 3).astype(np.int32)


def run_all(q, k, v, **kw) -> OracleResult:
    qb = _bits(q)
    B, Hq, N, _ = qb.shape
    return run_units(qb, k, v, all_units(B, Hq, N, kw.get("group_rows", 0) or 32), **kw)
