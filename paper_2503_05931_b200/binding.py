"""Thin Python binding of the AED decoder C ABI (``include/aed_dec.h``).

Argument marshalling only: every arithmetic step runs in the CUDA library.  PyTorch is used for
device memory and streams.  The shared library is built in-tree by ``build_ext.build()``; importing
this module without it fails loudly (there is no CPU fallback).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AED_DEC_LIB") or os.path.join(_HERE, "libaed_dec.so")   # AED_DEC_LIB: debug builds

AED_OK, AED_ERR_INVALID_ARG, AED_ERR_CAPACITY, AED_ERR_STATE = 0, -1, -2, -3
AED_ERR_CUDA, AED_ERR_TIMEOUT, AED_ERR_UNSUPPORTED = -4, -5, -6
AED_DTYPE_F32, AED_DTYPE_BF16 = 0, 1
AED_CROSS_KV_DTYPE, AED_CROSS_KV_E4M3 = 0, 1

EXPORTED_SYMBOLS = [
    "aed_dec_workspace_bytes", "aed_dec_create", "aed_dec_precompute_cross_kv", "aed_dec_step",
    "aed_dec_greedy_decode", "aed_dec_sync_status", "aed_dec_launch_count", "aed_dec_destroy",
    "aed_dec_last_error", "aed_dec_create_error", "aed_dec_profile_enable", "aed_dec_profile_read",
    "aed_dec_step_static_scratch", "aed_dec_static_scratch_bytes", "aed_dec_status_of_error_word", "aed_dec_prefill",
    "aed_dec_open_slots", "aed_dec_admit", "aed_dec_greedy_steps", "aed_dec_decode_stream",
]

_GLOBAL_FIELDS = ["embed", "final_ln_g", "final_ln_b", "w_out", "b_out"]
_LAYER_FIELDS = ["ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                 "ln2_g", "ln2_b", "w_q_c", "b_q_c", "w_kv_c", "b_kv_c", "w_o_c", "b_o_c",
                 "ln3_g", "ln3_b", "w_ff1", "b_ff1", "w_ff2", "b_ff2"]


class AedConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "d_ffn", "vocab", "d_enc", "dtype",
                                         "max_batch", "max_total_enc_frames", "max_enc_len", "max_dec_len",
                                         "bos_id", "eos_id")] + \
               [("ln_eps", C.c_float), ("cross_kv_format", C.c_int32), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("stream", C.c_void_p)]


class AedWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _GLOBAL_FIELDS] + [(n, C.POINTER(C.c_void_p)) for n in _LAYER_FIELDS]


class AedError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"aed_dec status {status}: {message}")
        self.status = status
        self.message = message


_lib: Optional[C.CDLL] = None


def load_library() -> C.CDLL:
    """Load the CUDA library; raises if it has not been built (no fallback of any kind)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with paper_2503_05931_b200.build_ext.build()")
    lib = C.CDLL(LIB_PATH)
    lib.aed_dec_workspace_bytes.restype = C.c_size_t
    lib.aed_dec_workspace_bytes.argtypes = [C.POINTER(AedConfig)]
    lib.aed_dec_create.restype = C.c_int
    lib.aed_dec_create.argtypes = [C.POINTER(AedConfig), C.POINTER(AedWeights), C.POINTER(C.c_void_p)]
    lib.aed_dec_precompute_cross_kv.restype = C.c_int
    lib.aed_dec_precompute_cross_kv.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32), C.c_int32]
    lib.aed_dec_step.restype = C.c_int
    lib.aed_dec_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.aed_dec_open_slots.restype = C.c_int
    lib.aed_dec_open_slots.argtypes = [C.c_void_p, C.c_int32]
    lib.aed_dec_admit.restype = C.c_int
    lib.aed_dec_admit.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
    lib.aed_dec_greedy_steps.restype = C.c_int
    lib.aed_dec_greedy_steps.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
    lib.aed_dec_decode_stream.restype = C.c_int
    lib.aed_dec_decode_stream.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                          C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_int64),
                                          C.POINTER(C.c_int64)]
    lib.aed_dec_prefill.restype = C.c_int
    lib.aed_dec_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    lib.aed_dec_step_static_scratch.restype = C.c_int
    lib.aed_dec_step_static_scratch.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.aed_dec_static_scratch_bytes.restype = C.c_size_t
    lib.aed_dec_static_scratch_bytes.argtypes = []
    lib.aed_dec_greedy_decode.restype = C.c_int
    lib.aed_dec_greedy_decode.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_void_p, C.c_void_p]
    lib.aed_dec_sync_status.restype = C.c_int
    lib.aed_dec_sync_status.argtypes = [C.c_void_p]
    lib.aed_dec_status_of_error_word.restype = C.c_int
    lib.aed_dec_status_of_error_word.argtypes = [C.c_int32]
    lib.aed_dec_launch_count.restype = C.c_int64
    lib.aed_dec_launch_count.argtypes = [C.c_void_p]
    lib.aed_dec_destroy.restype = None
    lib.aed_dec_destroy.argtypes = [C.c_void_p]
    lib.aed_dec_last_error.restype = C.c_char_p
    lib.aed_dec_last_error.argtypes = [C.c_void_p]
    lib.aed_dec_create_error.restype = C.c_char_p
    lib.aed_dec_create_error.argtypes = []
    lib.aed_dec_profile_enable.restype = C.c_int
    lib.aed_dec_profile_enable.argtypes = [C.c_void_p, C.c_int32]
    lib.aed_dec_profile_read.restype = C.c_int32
    lib.aed_dec_profile_read.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_char_p), C.POINTER(C.c_double),
                                         C.POINTER(C.c_int64)]
    _lib = lib
    return lib


def make_config(model: Dict[str, int], dtype: str, *, max_batch: int, max_total_enc_frames: int, max_enc_len: int,
                max_dec_len: int, bos_id: int = 1, eos_id: int = -1, ln_eps: float = 1e-5,
                cross_kv_e4m3: bool = False) -> AedConfig:
    return AedConfig(model["n_layers"], model["d_model"], model["n_heads"], model["d_ffn"], model["vocab"],
                     model["d_enc"], AED_DTYPE_BF16 if dtype == "bf16" else AED_DTYPE_F32, max_batch,
                     max_total_enc_frames, max_enc_len, max_dec_len, bos_id, eos_id, ln_eps,
                     AED_CROSS_KV_E4M3 if cross_kv_e4m3 else AED_CROSS_KV_DTYPE, None, 0, None)


def workspace_bytes(cfg: AedConfig) -> int:
    return int(load_library().aed_dec_workspace_bytes(C.byref(cfg)))


class Decoder:
    """One decoder handle: owns the device workspace and keeps the weight tensors alive.

    ``weights`` maps tensor names to float32 numpy arrays (per-layer tensors: one array per layer), as made
    by ``workloads.draw_weights``; they are uploaded in the configured dtype.  A missing / None bias = no bias.
    """

    def __init__(self, model: Dict[str, int], weights: Dict[str, object], dtype: str = "fp32", *, max_batch: int,
                 max_total_enc_frames: int, max_enc_len: int, max_dec_len: int, bos_id: int = 1, eos_id: int = -1,
                 ln_eps: float = 1e-5, device: str = "cuda:0", stream=None, cross_kv_e4m3: bool = False):
        import torch
        self._torch = torch
        self.lib = load_library()
        self.model = dict(model)
        self.dtype = dtype
        self.device = torch.device(device)
        self.tdtype = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.max_batch, self.max_dec_len = int(max_batch), int(max_dec_len)
        self.handle = C.c_void_p()
        self.cfg = make_config(model, dtype, max_batch=max_batch, max_total_enc_frames=max_total_enc_frames,
                               max_enc_len=max_enc_len, max_dec_len=max_dec_len, bos_id=bos_id, eos_id=eos_id,
                               ln_eps=ln_eps, cross_kv_e4m3=cross_kv_e4m3)
        need = int(self.lib.aed_dec_workspace_bytes(C.byref(self.cfg)))
        if need == 0:
            # let create produce the precise error
            need = 256
        with torch.cuda.device(self.device):
            self.stream = stream if stream is not None else torch.cuda.current_stream()
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
            self.cfg.workspace = self.workspace.data_ptr()
            self.cfg.workspace_bytes = need
            self.cfg.stream = self.stream.cuda_stream
            self._tensors = []
            w = AedWeights()
            nl = model["n_layers"]
            for name in _GLOBAL_FIELDS:
                arr = weights.get(name)
                setattr(w, name, self._upload(arr) if arr is not None else None)
            self._ptr_arrays = []
            for name in _LAYER_FIELDS:
                arrs = weights.get(name)
                if arrs is None:
                    setattr(w, name, C.POINTER(C.c_void_p)())
                    continue
                ptrs = (C.c_void_p * nl)(*[self._upload(a) for a in arrs])
                self._ptr_arrays.append(ptrs)
                setattr(w, name, C.cast(ptrs, C.POINTER(C.c_void_p)))
            self.weights_struct = w
            rc = self.lib.aed_dec_create(C.byref(self.cfg), C.byref(w), C.byref(self.handle))
        if rc != AED_OK:
            self.handle = C.c_void_p()
            raise AedError(rc, self.lib.aed_dec_create_error().decode())
        self.batch = 0

    def _upload(self, arr) -> int:
        torch = self._torch
        t = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(self.device).to(self.tdtype).contiguous()
        self._tensors.append(t)
        return t.data_ptr()

    def _check(self, rc: int) -> None:
        if rc != AED_OK:
            raise AedError(rc, self.lib.aed_dec_last_error(self.handle).decode())

    # ---- the five calls -----------------------------------------------------------------------------
    def precompute_cross_kv(self, enc_packed, enc_lens: Sequence[int]) -> None:
        """enc_packed: device tensor [sum(enc_lens), d_enc] in the configured dtype."""
        lens = np.ascontiguousarray(enc_lens, dtype=np.int32)
        assert enc_packed.is_cuda and enc_packed.dtype == self.tdtype and enc_packed.is_contiguous()
        self._enc_keepalive = enc_packed
        self._check(self.lib.aed_dec_precompute_cross_kv(self.handle, enc_packed.data_ptr(),
                                                         lens.ctypes.data_as(C.POINTER(C.c_int32)), len(lens)))
        self.batch = len(lens)

    def step(self, tokens_in, active=None, logits_out=None, next_out=None) -> None:
        """All arguments are device tensors: tokens_in int32 [B], active uint8 [B] or None,
        logits_out float32 [B, V] or None, next_out int32 [B] or None."""
        ptr = lambda t: t.data_ptr() if t is not None else None
        self._check(self.lib.aed_dec_step(self.handle, ptr(tokens_in), ptr(active), ptr(logits_out), ptr(next_out)))

    def prefill(self, prompt, logits_out=None, next_out=None) -> None:
        """prompt: device int32 tensor [batch, prompt_len]; logits_out / next_out describe the last prompt position."""
        assert prompt.is_cuda and prompt.dtype == self._torch.int32 and prompt.is_contiguous() and prompt.dim() == 2
        ptr = lambda t: t.data_ptr() if t is not None else None
        self._check(self.lib.aed_dec_prefill(self.handle, prompt.data_ptr(), int(prompt.shape[1]), ptr(logits_out), ptr(next_out)))

    def step_static_scratch(self, tokens_in, active=None, logits_out=None, next_out=None) -> None:
        """``step`` with the attention scratch in the library's built-in device array (for callers that
        cannot allocate device memory); same arguments as ``step``."""
        ptr = lambda t: t.data_ptr() if t is not None else None
        self._check(self.lib.aed_dec_step_static_scratch(self.handle, ptr(tokens_in), ptr(active), ptr(logits_out),
                                                         ptr(next_out)))

    def greedy_decode(self, max_len: Sequence[int], tokens_out=None, out_lens=None):
        torch = self._torch
        ml = np.ascontiguousarray(max_len, dtype=np.int32)
        if tokens_out is None:
            tokens_out = torch.empty((len(ml), self.max_dec_len), dtype=torch.int32, device=self.device)
        if out_lens is None:
            out_lens = torch.empty(len(ml), dtype=torch.int32, device=self.device)
        self._check(self.lib.aed_dec_greedy_decode(self.handle, ml.ctypes.data_as(C.POINTER(C.c_int32)),
                                                   tokens_out.data_ptr(), out_lens.data_ptr()))
        return tokens_out, out_lens

    def open_slots(self, slots: int) -> None:
        self._check(self.lib.aed_dec_open_slots(self.handle, int(slots)))
        self.batch = int(slots)

    def admit(self, slot: int, enc, max_len: int, out_lens=None) -> None:
        """enc: device tensor [enc_len, d_enc] in the handle's dtype (a contiguous slice of a packed buffer will do)."""
        assert enc.is_cuda and enc.dtype == self.tdtype and enc.is_contiguous() and enc.dim() == 2
        self._check(self.lib.aed_dec_admit(self.handle, int(slot), enc.data_ptr(), int(enc.shape[0]), int(max_len),
                                           out_lens.data_ptr() if out_lens is not None else None))

    def greedy_steps(self, n_steps: int, tokens_out, out_lens) -> int:
        done = C.c_int32(0)
        self._check(self.lib.aed_dec_greedy_steps(self.handle, int(n_steps), tokens_out.data_ptr(), out_lens.data_ptr(),
                                                  C.byref(done)))
        return int(done.value)

    def decode_stream(self, enc_packed, enc_lens, max_lens, slots: int, *, order=None, poll_steps: int = 8,
                      tokens_out=None, out_lens=None):
        """tokens_out / out_lens: pinned host tensors int32 [n, max_dec_len] / [n] (allocated if None).
        Returns (tokens_out, out_lens, steps, row_steps)."""
        torch = self._torch
        assert enc_packed.is_cuda and enc_packed.dtype == self.tdtype and enc_packed.is_contiguous()
        el = np.ascontiguousarray(enc_lens, dtype=np.int32)
        ml = np.ascontiguousarray(max_lens, dtype=np.int32)
        n = len(el)
        assert len(ml) == n and int(el.sum()) == enc_packed.shape[0]
        od = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
        if tokens_out is None:
            tokens_out = torch.empty((n, self.max_dec_len), dtype=torch.int32).pin_memory()
        if out_lens is None:
            out_lens = torch.zeros(n, dtype=torch.int32).pin_memory()
        assert not tokens_out.is_cuda and not out_lens.is_cuda and tokens_out.is_contiguous() and out_lens.is_contiguous()
        steps, row_steps = C.c_int64(0), C.c_int64(0)
        i32p = C.POINTER(C.c_int32)
        self._check(self.lib.aed_dec_decode_stream(self.handle, enc_packed.data_ptr(), el.ctypes.data_as(i32p), ml.ctypes.data_as(i32p),
                                                   od.ctypes.data_as(i32p) if od is not None else None, n, int(slots),
                                                   int(poll_steps), tokens_out.data_ptr(), out_lens.data_ptr(),
                                                   C.byref(steps), C.byref(row_steps)))
        self.batch = int(slots)
        return tokens_out, out_lens, int(steps.value), int(row_steps.value)

    def sync_status(self) -> None:
        self._check(self.lib.aed_dec_sync_status(self.handle))

    def launch_count(self) -> int:
        return int(self.lib.aed_dec_launch_count(self.handle))

    def profile_pass(self, fn):
        """Run ``fn(False)`` once with per-launch CUDA events on; returns {family: {"ms", "launches"}}."""
        self._check(self.lib.aed_dec_profile_enable(self.handle, 1))
        try:
            fn(False)
            names = (C.c_char_p * 64)()
            ms = (C.c_double * 64)()
            cnt = (C.c_int64 * 64)()
            n = self.lib.aed_dec_profile_read(self.handle, 64, names, ms, cnt)
            if n < 0:
                self._check(n)
            return {names[i].decode(): {"ms": float(ms[i]), "launches": int(cnt[i])} for i in range(n)}
        finally:
            self._check(self.lib.aed_dec_profile_enable(self.handle, 0))

    def close(self) -> None:
        if getattr(self, "handle", None) and self.handle.value:
            self.lib.aed_dec_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- convenience for tests and benchmarks (marshalling only) ---------------------------------------
    def upload_encoder(self, enc: np.ndarray):
        torch = self._torch
        return torch.from_numpy(np.ascontiguousarray(enc, dtype=np.float32)).to(self.device).to(self.tdtype).contiguous()


def decoder_for_workload(w, *, max_batch: Optional[int] = None, max_dec_len: Optional[int] = None,
                         device: str = "cuda:0", eos_id: Optional[int] = None, cross_kv_e4m3: bool = False) -> Decoder:
    """A Decoder sized for one seeded workload (see ``workloads.make_workload``)."""
    return Decoder(w.model, w.weights, w.dtype, max_batch=max_batch or w.batch,
                   max_total_enc_frames=int(w.enc_lens.sum()), max_enc_len=int(w.enc_lens.max()),
                   max_dec_len=max_dec_len or int(w.dec_lens.max()), bos_id=w.bos_id,
                   eos_id=w.eos_id if eos_id is None else eos_id, ln_eps=w.ln_eps, device=device, cross_kv_e4m3=cross_kv_e4m3)
