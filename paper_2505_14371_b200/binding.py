"""Thin ctypes binding of liblq.so: argument marshalling only.

Every step of the hot path runs inside the CUDA library; this module only converts torch
tensors to raw device pointers and passes the current CUDA stream.  Function names mirror
the C entry points declared in include/lq.h.  There is no CPU fallback: if the library is
missing, importing it raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblq.so")

NUM_BINS = 386
HIST_STRIDE = 512
STATUS_ZERO_NORM = 1
STATUS_NONFINITE = 2
STEP_AUTO = 0xFFFFFFFF          # lq_quantize_pack: take the step index from the plan's device-side iteration counter

EXPORTS = ["lq_plan_create", "lq_plan_destroy", "lq_plan_padded_elems", "lq_plan_packed_words",
           "lq_plan_layer_info", "lq_set_norm_scope", "lq_plan_norm_count", "lq_layer_weights", "lq_set_worker_range", "lq_message_modified", "lq_side_data_export",
           "lq_side_data_import", "lq_set_levels", "lq_get_levels", "lq_layer_norms",
           "lq_quantize_pack", "lq_fit_levels", "lq_fit_levels_shared", "lq_decode_aggregate", "qoda_init", "qoda_step",
           "qoda_get_scalars", "lq_code_build", "lq_code_universal", "lq_code_set", "lq_code_get", "lq_plan_blocks", "lq_entropy_encode",
           "lq_entropy_decode", "lq_entropy_status", "lq_level_probabilities", "lq_symbol_counts", "qoda_set_alt_rates", "qoda_set_average", "qoda_get_alt_scalars", "lq_get_statistics", "lq_vector_norm_static", "lq_profile_enable",
           "lq_profile_read",
           "lq_error_string", "lq_last_error"]
KERNEL_NAMES = ["norm_partial", "norm_finalize", "quantize_pack", "stat_finalize", "qoda_scalars",
                "decode", "fit", "alt_finalize", "average", "block_live"]


class LqError(RuntimeError):
    pass


_lib = None


def load_library() -> C.CDLL:
    """dlopen liblq.so and declare the C signatures.  Raises if the library was not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise LqError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_14371_b200.build` "
                      "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, u32, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64
    L.lq_plan_create.argtypes = [C.POINTER(vp), i32, C.POINTER(i64), C.POINTER(i32), i32, i32, u64]
    L.lq_plan_destroy.argtypes = [vp]
    L.lq_plan_padded_elems.argtypes = [vp]; L.lq_plan_padded_elems.restype = i64
    L.lq_plan_packed_words.argtypes = [vp]; L.lq_plan_packed_words.restype = i64
    L.lq_plan_layer_info.argtypes = [vp, i32, C.POINTER(i64), C.POINTER(i64), C.POINTER(i32)]
    L.lq_set_norm_scope.argtypes = [vp, i32]
    L.lq_plan_norm_count.argtypes = [vp]
    L.lq_plan_norm_count.restype = i64
    L.lq_layer_weights.argtypes = [vp, vp]
    L.lq_set_worker_range.argtypes = [vp, i32, i32]
    L.lq_message_modified.argtypes = [vp]
    L.lq_side_data_export.argtypes = [vp, vp, vp, vp, vp]
    L.lq_side_data_import.argtypes = [vp, vp, vp, vp, vp]
    L.lq_set_levels.argtypes = [vp, i32, C.POINTER(C.c_float), i32]
    L.lq_get_levels.argtypes = [vp, i32, C.POINTER(C.c_float), i32]
    L.lq_layer_norms.argtypes = [vp, vp, vp, vp]
    L.lq_quantize_pack.argtypes = [vp, vp, u32, vp, vp, vp, vp, vp, vp]
    L.lq_fit_levels.argtypes = [vp, vp, vp, i32, vp]
    L.lq_fit_levels_shared.argtypes = [vp, vp, vp, i32, C.POINTER(i32), vp]
    L.lq_decode_aggregate.argtypes = [vp, vp, vp, vp, vp]
    L.qoda_init.argtypes = [vp, vp, vp, vp, vp]
    L.qoda_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.qoda_get_scalars.argtypes = [vp, C.POINTER(i64), C.POINTER(C.c_double), C.POINTER(C.c_double)]
    u8p = C.POINTER(C.c_uint8)
    L.lq_code_build.argtypes = [C.POINTER(C.c_double), i32, u8p]
    L.lq_code_universal.argtypes = [i32, u8p]
    L.lq_code_set.argtypes = [vp, i32, u8p, i32]
    L.lq_code_get.argtypes = [vp, i32, u8p, i32]
    L.lq_plan_blocks.argtypes = [vp]; L.lq_plan_blocks.restype = i64
    L.lq_entropy_encode.argtypes = [vp, vp, vp, i64, vp, vp, vp]
    L.lq_entropy_decode.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    L.lq_entropy_status.argtypes = [vp, C.POINTER(u32)]
    L.lq_level_probabilities.argtypes = [vp, vp, vp, i32, i32, vp, vp]
    L.lq_symbol_counts.argtypes = [vp, vp, vp, vp]
    L.qoda_set_alt_rates.argtypes = [vp, C.c_double]
    L.qoda_set_average.argtypes = [vp, vp, vp]
    L.qoda_get_alt_scalars.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.lq_get_statistics.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(u32)]
    L.lq_vector_norm_static.argtypes = [vp, i64, i32, vp, vp, vp]
    L.lq_profile_enable.argtypes = [vp, i32]
    L.lq_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
    L.lq_error_string.argtypes = [C.c_int]; L.lq_error_string.restype = C.c_char_p
    L.lq_last_error.argtypes = []; L.lq_last_error.restype = C.c_char_p
    for name in EXPORTS:
        getattr(L, name)              # raises AttributeError if the library lacks an entry point
    _lib = L
    return L


def _check(code: int) -> None:
    if code != 0:
        L = load_library()
        raise LqError(f"{L.lq_error_string(code).decode()} ({code}): {L.lq_last_error().decode()}")


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise LqError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise LqError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def lq_vector_norm_static(v: torch.Tensor, q: int, norm_out: torch.Tensor,
                          status_out: Optional[torch.Tensor] = None) -> None:
    """L^q norm of the fp32 device vector `v` into norm_out[0] through the library's fixed scratch
    array: no plan and no allocation below this call.  For callers whose device memory is all
    spoken for, or who cannot afford the synchronisation an allocation implies.  Calls must not
    overlap on the GPU (they share the scratch)."""
    _check(load_library().lq_vector_norm_static(_ptr(v, torch.float32), v.numel(), int(q),
                                                _ptr(norm_out, torch.float32), _ptr(status_out, torch.int32),
                                                _stream()))


def lq_code_build(weights) -> List[int]:
    """Huffman word lengths for the given symbol weights (host only)."""
    n = len(weights)
    w = (C.c_double * n)(*[float(x) for x in weights]); out = (C.c_uint8 * n)()
    _check(load_library().lq_code_build(w, n, out))
    return list(out)


def lq_code_universal(n: int) -> List[int]:
    """Word lengths of Elias' recursive code for level indices 0..n-1 (host only)."""
    out = (C.c_uint8 * n)()
    _check(load_library().lq_code_universal(int(n), out))
    return list(out)


class Plan:
    """Owns one lq_plan.  Methods carry the names of the C entry points."""

    def __init__(self, layer_sizes: Sequence[int], bits, q: int, num_workers: int, seed: int):
        L = load_library()
        n = len(layer_sizes)
        if isinstance(bits, int):
            bits = [bits] * n
        self.layer_sizes = [int(s) for s in layer_sizes]
        self.bits = [int(b) for b in bits]
        self.q, self.num_workers, self.seed = int(q), int(num_workers), int(seed)
        sizes = (C.c_int64 * max(n, 1))(*self.layer_sizes)
        bb = (C.c_int32 * max(n, 1))(*self.bits)
        h = C.c_void_p()
        _check(L.lq_plan_create(C.byref(h), n, sizes, bb, self.q, self.num_workers, C.c_uint64(self.seed)))
        self._h = h
        self.num_layers = n
        self.padded_elems = int(L.lq_plan_padded_elems(h))
        self.packed_words = int(L.lq_plan_packed_words(h))
        self.elem_offsets: List[int] = []
        self.word_offsets: List[int] = []
        for m in range(n):
            e, w, nl = C.c_int64(), C.c_int64(), C.c_int32()
            _check(L.lq_plan_layer_info(h, m, C.byref(e), C.byref(w), C.byref(nl)))
            self.elem_offsets.append(e.value); self.word_offsets.append(w.value)

    def close(self) -> None:
        if getattr(self, "_h", None):
            load_library().lq_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def lq_set_norm_scope(self, scope: str) -> None:
        """"layer" (default), "global" (one norm over the worker's whole vector) or "bucket" (one norm per 128
        consecutive coordinates of a layer; norms buffers then have lq_plan_norm_count() values per worker)."""
        _check(load_library().lq_set_norm_scope(self._h, {"layer": 0, "global": 1, "bucket": 2}[scope]))

    def lq_message_modified(self) -> None:
        _check(load_library().lq_message_modified(self._h))

    def lq_set_worker_range(self, first_worker: int, count: int) -> None:
        _check(load_library().lq_set_worker_range(self._h, int(first_worker), int(count)))

    def lq_side_data_export(self, sq_diff=None, layer_weight=None, flags=None) -> None:
        _check(load_library().lq_side_data_export(self._h, _ptr(sq_diff, torch.float64), _ptr(layer_weight, torch.float32),
                                                  _ptr(flags, torch.int32), _stream()))

    def lq_side_data_import(self, sq_diff=None, layer_weight=None, flags=None) -> None:
        _check(load_library().lq_side_data_import(self._h, _ptr(sq_diff, torch.float64), _ptr(layer_weight, torch.float32),
                                                  _ptr(flags, torch.int32), _stream()))

    def lq_plan_norm_count(self) -> int:
        n = int(load_library().lq_plan_norm_count(self._h))
        if n < 0:
            _check(n)
        return n

    def lq_layer_weights(self) -> torch.Tensor:
        out = torch.empty((self.num_workers, max(self.num_layers, 1)), dtype=torch.float32)
        _check(load_library().lq_layer_weights(self._h, out.data_ptr()))
        return out[:, :self.num_layers]

    # ---- levels -------------------------------------------------------------------------
    def lq_set_levels(self, layer: int, levels) -> None:
        arr = (C.c_float * len(levels))(*[float(x) for x in levels])
        _check(load_library().lq_set_levels(self._h, layer, arr, len(levels)))

    def lq_get_levels(self, layer: int) -> List[float]:
        n = 1 << self.bits[layer]
        arr = (C.c_float * n)()
        _check(load_library().lq_get_levels(self._h, layer, arr, n))
        return list(arr)

    # ---- hot path -----------------------------------------------------------------------
    def lq_layer_norms(self, grads: torch.Tensor, norms: torch.Tensor) -> None:
        _check(load_library().lq_layer_norms(self._h, _ptr(grads, torch.float32), _ptr(norms, torch.float32),
                                             _stream()))

    def lq_quantize_pack(self, grads, step: int, packed, norms, hist=None, prev_packed=None,
                         prev_norms=None) -> None:
        _check(load_library().lq_quantize_pack(
            self._h, _ptr(grads, torch.float32), C.c_uint32(step & 0xFFFFFFFF), _ptr(packed, torch.int32),
            _ptr(norms, torch.float32), _ptr(hist, torch.int32), _ptr(prev_packed, torch.int32),
            _ptr(prev_norms, torch.float32), _stream()))

    def lq_fit_levels(self, hist, norms, num_samples: int) -> None:
        _check(load_library().lq_fit_levels(self._h, _ptr(hist, torch.int32), _ptr(norms, torch.float32),
                                            num_samples, _stream()))

    def lq_fit_levels_shared(self, hist, norms, num_samples: int, layer_type: Sequence[int]) -> None:
        ids = (C.c_int32 * max(self.num_layers, 1))(*[int(t) for t in layer_type])
        _check(load_library().lq_fit_levels_shared(self._h, _ptr(hist, torch.int32), _ptr(norms, torch.float32),
                                                   num_samples, ids, _stream()))

    def lq_decode_aggregate(self, packed, norms, gbar) -> None:
        _check(load_library().lq_decode_aggregate(self._h, _ptr(packed, torch.int32), _ptr(norms, torch.float32),
                                                  _ptr(gbar, torch.float32), _stream()))

    def qoda_init(self, X1, Y, Xhalf) -> None:
        _check(load_library().qoda_init(self._h, _ptr(X1, torch.float32), _ptr(Y, torch.float32),
                                        _ptr(Xhalf, torch.float32), _stream()))

    def qoda_step(self, packed, norms, X1, Y, Xhalf, X=None, gbar=None) -> None:
        _check(load_library().qoda_step(self._h, _ptr(packed, torch.int32), _ptr(norms, torch.float32),
                                        _ptr(X1, torch.float32), _ptr(Y, torch.float32),
                                        _ptr(Xhalf, torch.float32), _ptr(X, torch.float32),
                                        _ptr(gbar, torch.float32), _stream()))

    def qoda_get_scalars(self):
        t, S, eta = C.c_int64(), C.c_double(), C.c_double()
        _check(load_library().qoda_get_scalars(self._h, C.byref(t), C.byref(S), C.byref(eta)))
        return t.value, S.value, eta.value

    def lq_level_probabilities(self, hist, norms, num_samples: int, probs, staged: bool = False) -> None:
        _check(load_library().lq_level_probabilities(self._h, _ptr(hist, torch.int32), _ptr(norms, torch.float32),
                                                     num_samples, 1 if staged else 0, _ptr(probs, torch.float64),
                                                     _stream()))

    def lq_symbol_counts(self, packed, counts) -> None:
        _check(load_library().lq_symbol_counts(self._h, _ptr(packed, torch.int32), _ptr(counts, torch.int32), _stream()))

    # ---- entropy stage --------------------------------------------------------------------
    def lq_code_set(self, layer: int, lengths) -> None:
        arr = (C.c_uint8 * len(lengths))(*[int(x) for x in lengths])
        _check(load_library().lq_code_set(self._h, layer, arr, len(lengths)))

    def lq_code_get(self, layer: int) -> List[int]:
        n = 1 << self.bits[layer]
        arr = (C.c_uint8 * n)()
        _check(load_library().lq_code_get(self._h, layer, arr, n))
        return list(arr)

    def lq_plan_blocks(self) -> int:
        return int(load_library().lq_plan_blocks(self._h))

    def lq_entropy_encode(self, packed, stream_words, block_offsets, run_offsets=None) -> None:
        _check(load_library().lq_entropy_encode(self._h, _ptr(packed, torch.int32), _ptr(stream_words, torch.int32),
                                                stream_words.shape[1], _ptr(block_offsets, torch.int32),
                                                _ptr(run_offsets, torch.int16), _stream()))

    def lq_entropy_decode(self, stream_words, block_offsets, packed, run_offsets=None) -> None:
        _check(load_library().lq_entropy_decode(self._h, _ptr(stream_words, torch.int32), stream_words.shape[1],
                                                _ptr(block_offsets, torch.int32), _ptr(run_offsets, torch.int16),
                                                _ptr(packed, torch.int32), _stream()))

    def empty_run_offsets(self, device="cuda"):
        """[K][blocks][8] int16 buffer for the run offsets of the entropy stage."""
        return torch.zeros((self.num_workers, self.lq_plan_blocks(), 8), dtype=torch.int16, device=device)

    def lq_entropy_status(self) -> int:
        flag = C.c_uint32(0)
        _check(load_library().lq_entropy_status(self._h, C.byref(flag)))
        return flag.value

    def qoda_set_average(self, xsum: Optional[torch.Tensor]) -> None:
        """Registers (or with None removes) the fp64 running sum of the half iterates; the tensor must stay alive."""
        _check(load_library().qoda_set_average(self._h, _ptr(xsum, torch.float64), _stream()))
        self._xsum = xsum

    def qoda_set_alt_rates(self, q_hat: float) -> None:
        _check(load_library().qoda_set_alt_rates(self._h, float(q_hat)))

    def qoda_get_alt_scalars(self):
        lam, mu, gamma = C.c_double(), C.c_double(), C.c_double()
        _check(load_library().qoda_get_alt_scalars(self._h, C.byref(lam), C.byref(mu), C.byref(gamma)))
        return lam.value, mu.value, gamma.value

    def lq_get_statistics(self):
        """Returns (sq_diff [K][L] float64, status [K][L] int) as torch CPU tensors."""
        K, Ln = self.num_workers, max(self.num_layers, 1)
        sq = (C.c_double * (K * Ln))(); fl = (C.c_uint32 * (K * Ln))()
        _check(load_library().lq_get_statistics(self._h, sq, fl))
        return (torch.tensor(list(sq), dtype=torch.float64).view(K, Ln)[:, : self.num_layers],
                torch.tensor(list(fl), dtype=torch.int64).view(K, Ln)[:, : self.num_layers])

    def lq_profile_enable(self, enable: bool) -> None:
        _check(load_library().lq_profile_enable(self._h, 1 if enable else 0))

    def lq_profile_read(self):
        """Returns {kernel name: (total ms, launches)} since the last read."""
        n = len(KERNEL_NAMES)
        ms = (C.c_double * n)(); cnt = (C.c_int64 * n)()
        _check(load_library().lq_profile_read(self._h, ms, cnt))
        return {KERNEL_NAMES[i]: (ms[i], cnt[i]) for i in range(n)}

    # ---- allocation helpers (device memory only; no arithmetic) ----------------------------
    def empty_packed(self, device="cuda") -> torch.Tensor:
        return torch.empty((self.num_workers, max(self.packed_words, 1)), dtype=torch.int32, device=device)

    def empty_norms(self, device="cuda") -> torch.Tensor:
        return torch.empty((self.num_workers, max(self.lq_plan_norm_count(), 1)), dtype=torch.float32, device=device)

    def zero_hist(self, device="cuda") -> torch.Tensor:
        return torch.zeros((self.num_workers, max(self.num_layers, 1), HIST_STRIDE), dtype=torch.int32,
                           device=device)
