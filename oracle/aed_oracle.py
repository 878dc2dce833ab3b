"""ctypes front end of the CPU checker (``aed_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does.  It shares nothing with the CUDA library: the C
source is compiled here with gcc into two shared objects, an fp64 one (the parity
reference) and an fp32 one (timed as the CPU baseline).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aed_oracle.c")
_LIBS: Dict[str, C.CDLL] = {}

_LAYER_FIELDS = ["ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                 "ln2_g", "ln2_b", "w_q_c", "b_q_c", "w_kv_c", "b_kv_c", "w_o_c", "b_o_c",
                 "ln3_g", "ln3_b", "w_ff1", "b_ff1", "w_ff2", "b_ff2"]
_GLOBAL_FIELDS = ["embed", "final_ln_g", "final_ln_b", "w_out", "b_out"]
_FP = C.POINTER(C.c_float)
_FPP = C.POINTER(_FP)


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "d_ffn", "vocab", "d_enc")] + \
               [("ln_eps", C.c_double), ("cross_kv_e4m3", C.c_int32)]


class _Weights(C.Structure):
    _fields_ = [(n, _FP) for n in _GLOBAL_FIELDS] + [(n, _FPP) for n in _LAYER_FIELDS]


class _Trace(C.Structure):
    _fields_ = [("self_probs", C.POINTER(C.c_double)), ("cross_probs", C.POINTER(C.c_double))]


def lib_path(precision: str) -> str:
    return os.path.join(_HERE, f"libaed_oracle_{precision}.so")


def build(force: bool = False) -> None:
    """Compile the fp64 and fp32 checker libraries with gcc (plain -O2, OpenMP over utterances only)."""
    for precision, real in (("f64", "double"), ("f32", "float")):
        out = lib_path(precision)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", f"-DORC_REAL={real}", _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)


def load_custom(tag: str, path: str) -> None:
    """Register another build of the checker under ``precision=tag`` (tests that plant mistakes use this)."""
    lib = C.CDLL(path)
    _set_signatures(lib)
    _LIBS[tag] = lib


def _set_signatures(lib: C.CDLL) -> None:
    lib.orc_decode.restype = C.c_int
    lib.orc_decode_full_recompute.restype = C.c_int
    lib.orc_decode_batch.restype = C.c_int
    lib.orc_argmax_f64.restype = C.c_int32
    lib.orc_real_bytes.restype = C.c_int


def _lib(precision: str) -> C.CDLL:
    if precision not in _LIBS:
        build()
        lib = C.CDLL(lib_path(precision))
        lib.orc_decode.restype = C.c_int
        lib.orc_decode_full_recompute.restype = C.c_int
        lib.orc_decode_batch.restype = C.c_int
        lib.orc_argmax_f64.restype = C.c_int32
        lib.orc_real_bytes.restype = C.c_int
        _LIBS[precision] = lib
    return _LIBS[precision]


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


class Model:
    """Decoder parameters marshalled for the C checker.  ``weights`` maps tensor names to float32
    arrays (per-layer tensors: a list with one array per layer); a missing/None bias means no bias."""

    def __init__(self, model: Dict[str, int], weights: Dict[str, object], ln_eps: float = 1e-5,
                 cross_kv_e4m3: bool = False):
        """cross_kv_e4m3: the cross-attention keys and values are rounded to the 8-bit format E4M3 when stored."""
        self.model = dict(model)
        self.cfg = _Config(model["n_layers"], model["d_model"], model["n_heads"], model["d_ffn"],
                           model["vocab"], model["d_enc"], float(ln_eps), 1 if cross_kv_e4m3 else 0)
        self._keep: List[object] = []
        w = _Weights()
        nl = model["n_layers"]
        for name in _GLOBAL_FIELDS:
            arr = weights.get(name)
            if arr is None:
                setattr(w, name, _FP())
            else:
                arr = _f32(arr)
                self._keep.append(arr)
                setattr(w, name, arr.ctypes.data_as(_FP))
        for name in _LAYER_FIELDS:
            arrs = weights.get(name)
            if arrs is None:
                setattr(w, name, _FPP())
                continue
            assert len(arrs) == nl, name
            ptrs = (_FP * nl)()
            for l in range(nl):
                arr = _f32(arrs[l])
                self._keep.append(arr)
                ptrs[l] = arr.ctypes.data_as(_FP)
            self._keep.append(ptrs)
            setattr(w, name, C.cast(ptrs, _FPP))
        self.w = w


def decode(model: Model, enc: np.ndarray, n_steps: int, *, forced: Optional[Sequence[int]] = None, bos: int = 1,
           want_logits: bool = True, precision: str = "f64", full_recompute: bool = False, trace: bool = False,
           eos: int = -1):
    """Decode one utterance.  Returns dict(next [L] int32, margin [L], logits [L, V] or None, len,
    and with trace=True self_probs [L, NL, H, L] and cross_probs [L, NL, H, T]).  With ``eos`` >= 0 the
    utterance ends with the step that emits it: ``len`` counts that token and ``next`` is -1 afterwards."""
    lib = _lib(precision)
    enc = _f32(enc)
    T, L, V = int(enc.shape[0]), int(n_steps), model.model["vocab"]
    assert enc.shape[1] == model.model["d_enc"]
    nxt = np.zeros(L, np.int32)
    margin = np.zeros(L, np.float64)
    logits = np.zeros((L, V), np.float64) if want_logits else None
    f_arr = None
    if forced is not None:
        f_arr = np.ascontiguousarray(forced, dtype=np.int32)
        assert f_arr.shape == (L,)
    fp = f_arr.ctypes.data_as(C.POINTER(C.c_int32)) if f_arr is not None else None
    lp = logits.ctypes.data_as(C.POINTER(C.c_double)) if logits is not None else None
    common = [C.byref(model.cfg), C.byref(model.w), enc.ctypes.data_as(_FP), C.c_int32(T), fp, C.c_int32(bos),
              C.c_int32(L), lp, nxt.ctypes.data_as(C.POINTER(C.c_int32)), margin.ctypes.data_as(C.POINTER(C.c_double))]
    out = dict(next=nxt, margin=margin, logits=logits)
    if full_recompute:
        assert eos < 0, "the brute-force decoder has no end-of-sequence rule"
        rc = lib.orc_decode_full_recompute(*common)
        out["len"] = L
    else:
        tr = None
        if trace:
            nl, h = model.model["n_layers"], model.model["n_heads"]
            out["self_probs"] = np.zeros((L, nl, h, L), np.float64)
            out["cross_probs"] = np.zeros((L, nl, h, T), np.float64)
            tr = _Trace(out["self_probs"].ctypes.data_as(C.POINTER(C.c_double)),
                        out["cross_probs"].ctypes.data_as(C.POINTER(C.c_double)))
        n_out = C.c_int32(0)
        rc = lib.orc_decode(*common, C.byref(tr) if tr is not None else None, C.c_int32(eos), C.byref(n_out))
        out["len"] = int(n_out.value)
    if rc != 0:
        raise RuntimeError(f"oracle decode failed (rc={rc})")
    return out


def decode_batch(model: Model, enc_packed: np.ndarray, enc_lens: Sequence[int], dec_lens: Sequence[int], *,
                 forced: Optional[np.ndarray] = None, bos: int = 1, want_logits: bool = False,
                 precision: str = "f64", n_threads: int = 0, eos: int = -1):
    """Decode utterances independently (OpenMP over utterances).  Returns dict(next [B, Lmax] int32 (-1 padded),
    margin [B, Lmax], logits: list of [L_u, V] arrays or None, lens [B] emitted tokens, threads)."""
    lib = _lib(precision)
    enc_packed = _f32(enc_packed)
    enc_lens = np.asarray(enc_lens, dtype=np.int64)
    lens = np.ascontiguousarray(dec_lens, dtype=np.int32)
    B, V = len(lens), model.model["vocab"]
    off = np.zeros(B + 1, np.int64)
    np.cumsum(enc_lens, out=off[1:])
    assert enc_packed.shape[0] == off[-1]
    stride = int(lens.max()) if B else 1
    nxt = np.full((B, stride), -1, np.int32)
    margin = np.zeros((B, stride), np.float64)
    loff = np.zeros(B + 1, np.int64)
    np.cumsum(lens, out=loff[1:])
    logits = np.zeros((int(loff[-1]), V), np.float64) if want_logits else None
    out_lens = np.zeros(B, np.int32)
    f_arr = None
    if forced is not None:
        f_arr = np.ascontiguousarray(forced, dtype=np.int32)
        assert f_arr.shape == (B, stride)
    rc = lib.orc_decode_batch(
        C.byref(model.cfg), C.byref(model.w), enc_packed.ctypes.data_as(_FP),
        off.ctypes.data_as(C.POINTER(C.c_int64)), C.c_int32(B),
        f_arr.ctypes.data_as(C.POINTER(C.c_int32)) if f_arr is not None else None, C.c_int32(stride), C.c_int32(bos),
        lens.ctypes.data_as(C.POINTER(C.c_int32)),
        logits.ctypes.data_as(C.POINTER(C.c_double)) if logits is not None else None,
        loff.ctypes.data_as(C.POINTER(C.c_int64)),
        nxt.ctypes.data_as(C.POINTER(C.c_int32)), margin.ctypes.data_as(C.POINTER(C.c_double)), C.c_int32(n_threads),
        C.c_int32(eos), out_lens.ctypes.data_as(C.POINTER(C.c_int32)))
    if rc < 0:
        raise RuntimeError("oracle batch decode failed")
    per_utt = [logits[loff[u]:loff[u + 1]] for u in range(B)] if logits is not None else None
    return dict(next=nxt, margin=margin, logits=per_utt, lens=out_lens, threads=int(rc))


def layernorm(x, g, b, eps: float = 1e-5, precision: str = "f64") -> np.ndarray:
    lib = _lib(precision)
    x = np.ascontiguousarray(x, dtype=np.float64)
    g, b = _f32(g), _f32(b)
    y = np.zeros_like(x)
    lib.orc_layernorm_f64(x.ctypes.data_as(C.POINTER(C.c_double)), g.ctypes.data_as(_FP), b.ctypes.data_as(_FP),
                          C.c_int(x.shape[0]), C.c_double(eps), y.ctypes.data_as(C.POINTER(C.c_double)))
    return y


def round_e4m3(x, precision: str = "f64") -> np.ndarray:
    """Element-wise rounding to the 8-bit format E4M3 as the checker stores cross-attention keys and values."""
    lib = _lib(precision)
    lib.orc_round_e4m3.restype = C.c_double
    lib.orc_round_e4m3.argtypes = [C.c_double]
    x = np.asarray(x, dtype=np.float64)
    return np.array([lib.orc_round_e4m3(float(v)) for v in x.ravel()], dtype=np.float64).reshape(x.shape)


def argmax(z, precision: str = "f64"):
    lib = _lib(precision)
    z = np.ascontiguousarray(z, dtype=np.float64)
    m = C.c_double(0.0)
    idx = lib.orc_argmax_f64(z.ctypes.data_as(C.POINTER(C.c_double)), C.c_int(z.shape[0]), C.byref(m))
    return int(idx), float(m.value)
