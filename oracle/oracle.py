"""ctypes front end of the CPU oracle (oracle/lq_oracle.c) plus the QODA reference loop.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg.  It never imports the CUDA package, and the CUDA package never
imports it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lq_oracle.c")
_SO = os.path.join(_HERE, "_lq_oracle.so")
NUM_BINS = 386
HIST_STRIDE = 512


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction, no fast-math)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared",
                               "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u32p, f32p = C.POINTER(C.c_uint8), C.POINTER(C.c_uint32), C.POINTER(C.c_float)
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_uniform.restype = C.c_float
        L.orc_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64]
        L.orc_layer_norm.restype = C.c_float
        L.orc_layer_norm.argtypes = [f32p, C.c_int64, C.c_int, C.POINTER(C.c_int)]
        L.orc_quantize_layer.argtypes = [f32p, C.c_int64, C.c_int64, C.c_float, f32p, C.c_int, C.c_uint64,
                                         C.c_uint32, C.c_uint32, C.c_uint32, u8p, u8p,
                                         C.POINTER(C.c_int64)]
        L.orc_packed_words.restype = C.c_int64
        L.orc_packed_words.argtypes = [C.c_int64, C.c_int]
        L.orc_pack_layer.argtypes = [u8p, u8p, C.c_int64, C.c_int, u32p]
        L.orc_unpack_layer.argtypes = [u32p, C.c_int64, C.c_int, u8p, u8p]
        L.orc_bin_edge.restype = C.c_double
        L.orc_bin_edge.argtypes = [C.c_int]
        L.orc_histogram_layer.argtypes = [f32p, C.c_int64, C.c_float, u32p]
        L.orc_fit_levels.restype = C.c_int
        L.orc_fit_levels.argtypes = [u32p, C.c_int64, f32p, C.c_int, C.c_int64, C.c_int, f32p]
        L.orc_fit_levels_shared.restype = C.c_int
        L.orc_fit_levels_shared.argtypes = [u32p, C.c_int64, f32p, C.POINTER(C.c_int64), C.c_int, C.c_int, f32p]
        L.orc_fit_objective.restype = C.c_double
        L.orc_fit_objective.argtypes = [u32p, C.c_int64, f32p, C.c_int, C.c_int64, f32p, C.c_int]
        L.orc_decode_layer.argtypes = [u8p, u8p, C.c_int64, C.c_float, f32p, f32p]
        L.orc_aggregate.argtypes = [f32p, C.c_int, C.c_int64, f32p]
        L.orc_sq_diff.restype = C.c_double
        L.orc_sq_diff.argtypes = [f32p, f32p, C.c_int64]
        L.orc_step_size.restype = C.c_double
        L.orc_step_size.argtypes = [C.c_double, C.c_double, C.c_int, f32p]
        L.orc_qoda_update.argtypes = [f32p, f32p, f32p, f32p, f32p, C.c_float, C.c_int64]
        L.orc_level_probabilities.restype = C.c_int
        L.orc_level_probabilities.argtypes = [u32p, C.c_int64, f32p, C.c_int, C.c_int64, f32p, C.c_int, C.POINTER(C.c_double)]
        L.orc_expected_code_length.restype = C.c_double
        L.orc_expected_code_length.argtypes = [C.POINTER(C.c_double), C.c_int, C.c_int64, C.POINTER(C.c_double)]
        L.orc_huffman_lengths.restype = C.c_int
        L.orc_huffman_lengths.argtypes = [C.POINTER(C.c_double), C.c_int, C.c_int, u8p]
        L.orc_canonical_codes.argtypes = [u8p, C.c_int, u32p]
        L.orc_entropy_encode_block.restype = C.c_int64
        L.orc_entropy_encode_block.argtypes = [u8p, u8p, C.c_int, u8p, u32p, u32p]
        L.orc_entropy_decode_block.restype = C.c_int64
        L.orc_entropy_decode_block.argtypes = [u32p, C.c_int, u8p, u32p, C.c_int, u8p, u8p]
        L.orc_alt_rates.argtypes = [C.c_double, C.c_double, C.c_double, f32p, f32p]
        L.orc_sq_norm.restype = C.c_double
        L.orc_sq_norm.argtypes = [f32p, C.c_int64]
        L.orc_qoda_update_rates.argtypes = [f32p, f32p, f32p, f32p, f32p, C.c_float, C.c_float, C.c_int64]
        L.orc_elias_omega.restype = C.c_int
        L.orc_elias_omega.argtypes = [C.c_uint64, C.c_char_p]
        L.orc_elias_omega_decode.restype = C.c_uint64
        L.orc_elias_omega_decode.argtypes = [C.c_char_p, C.POINTER(C.c_int)]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray], ty):
    return None if a is None else a.ctypes.data_as(C.POINTER(ty))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


# --------------------------------------------------------------------------- primitives
def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> List[int]:
    c = np.array(ctr, dtype=np.uint32); k = np.array(key, dtype=np.uint32)
    o = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(o, C.c_uint32))
    return [int(x) for x in o]


def uniform(seed: int, step: int, worker: int, layer: int, index: int) -> float:
    return float(lib().orc_uniform(seed, step, worker, layer, index))


def layer_norm(v: np.ndarray, q: int):
    """Returns (fp32 norm, status) with status 0 ok / 1 zero / 2 non-finite."""
    v = _f32(v); st = C.c_int(0)
    n = lib().orc_layer_norm(_p(v, C.c_float), v.size, q, C.byref(st))
    return np.float32(n), st.value


def quantize_layer(v, norm, levels, seed, step, worker, layer, first_index=0):
    """Returns (idx u8[d], sign u8[d], near-threshold count) for coordinates
    first_index .. first_index+len(v)-1 of the layer."""
    v = _f32(v); levels = _f32(levels)
    idx = np.zeros(v.size, np.uint8); sg = np.zeros(v.size, np.uint8); near = C.c_int64(0)
    lib().orc_quantize_layer(_p(v, C.c_float), v.size, first_index, C.c_float(float(norm)), _p(levels, C.c_float),
                             levels.size, seed, step, worker, layer, _p(idx, C.c_uint8),
                             _p(sg, C.c_uint8), C.byref(near))
    return idx, sg, near.value


def packed_words(d: int, b: int) -> int:
    return int(lib().orc_packed_words(d, b))


def pack_layer(idx: np.ndarray, sign: np.ndarray, b: int) -> np.ndarray:
    idx = np.ascontiguousarray(idx, np.uint8); sign = np.ascontiguousarray(sign, np.uint8)
    w = np.zeros(packed_words(idx.size, b), np.uint32)
    lib().orc_pack_layer(_p(idx, C.c_uint8), _p(sign, C.c_uint8), idx.size, b, _p(w, C.c_uint32))
    return w


def unpack_layer(words: np.ndarray, d: int, b: int):
    words = np.ascontiguousarray(words, np.uint32)
    assert words.size >= packed_words(d, b)
    idx = np.zeros(d, np.uint8); sg = np.zeros(d, np.uint8)
    lib().orc_unpack_layer(_p(words, C.c_uint32), d, b, _p(idx, C.c_uint8), _p(sg, C.c_uint8))
    return idx, sg


def bin_edge(i: int) -> float:
    return float(lib().orc_bin_edge(i))


def histogram_layer(v, norm) -> np.ndarray:
    v = _f32(v); h = np.zeros(HIST_STRIDE, np.uint32)
    lib().orc_histogram_layer(_p(v, C.c_float), v.size, C.c_float(float(norm)), _p(h, C.c_uint32))
    return h


def fit_levels(hist: np.ndarray, norms, d: int, n: int):
    """hist [Z][stride] u32, norms [Z] fp32 -> (levels fp32[n] or None if no usable mass)."""
    hist = np.ascontiguousarray(hist, np.uint32).reshape(len(norms), -1); norms = _f32(norms)
    out = np.zeros(n, np.float32)
    ok = lib().orc_fit_levels(_p(hist, C.c_uint32), hist.shape[1], _p(norms, C.c_float),
                              norms.size, d, n, _p(out, C.c_float))
    return out if ok else None


def fit_levels_shared(hist: np.ndarray, norms, sizes, n: int):
    """One sequence for a type: hist [S][stride], norms [S], sizes [S] over all (sample, member layer) pairs."""
    norms = _f32(norms); sizes = np.ascontiguousarray(sizes, np.int64)
    hist = np.ascontiguousarray(hist, np.uint32).reshape(norms.size, -1)
    out = np.zeros(n, np.float32)
    ok = lib().orc_fit_levels_shared(_p(hist, C.c_uint32), hist.shape[1], _p(norms, C.c_float), _p(sizes, C.c_int64),
                                     norms.size, n, _p(out, C.c_float))
    return out if ok else None


def fit_objective(hist: np.ndarray, norms, d: int, levels) -> float:
    hist = np.ascontiguousarray(hist, np.uint32).reshape(len(norms), -1); norms = _f32(norms)
    levels = _f32(levels)
    return float(lib().orc_fit_objective(_p(hist, C.c_uint32), hist.shape[1], _p(norms, C.c_float),
                                         norms.size, d, _p(levels, C.c_float), levels.size))


def decode_layer(idx, sign, norm, levels) -> np.ndarray:
    idx = np.ascontiguousarray(idx, np.uint8); sign = np.ascontiguousarray(sign, np.uint8)
    levels = _f32(levels); out = np.zeros(idx.size, np.float32)
    lib().orc_decode_layer(_p(idx, C.c_uint8), _p(sign, C.c_uint8), idx.size, C.c_float(float(norm)),
                           _p(levels, C.c_float), _p(out, C.c_float))
    return out


def aggregate(decoded: np.ndarray) -> np.ndarray:
    decoded = _f32(decoded); K, d = decoded.shape
    out = np.zeros(d, np.float32)
    lib().orc_aggregate(_p(decoded, C.c_float), K, d, _p(out, C.c_float))
    return out


def sq_diff(cur: np.ndarray, prev: Optional[np.ndarray]) -> float:
    cur = _f32(cur); prev = None if prev is None else _f32(prev)
    return float(lib().orc_sq_diff(_p(cur, C.c_float), _p(prev, C.c_float), cur.size))


def step_size(S_prev: float, sum_sq: float, K: int):
    eta = C.c_float(0)
    S = lib().orc_step_size(S_prev, sum_sq, K, C.byref(eta))
    return float(S), np.float32(eta.value)


def qoda_update(gbar, X1, Y, Xhalf, X, eta) -> None:
    """In place on Y, Xhalf (and X when given); all contiguous fp32 arrays of one length."""
    lib().orc_qoda_update(_p(gbar, C.c_float), _p(X1, C.c_float), _p(Y, C.c_float),
                          _p(Xhalf, C.c_float), _p(X, C.c_float), C.c_float(float(eta)), gbar.size)


def level_probabilities(hist: np.ndarray, norms, d: int, levels) -> np.ndarray:
    """Probability of each level being emitted, from the merged histogram (Appendix, coding framework)."""
    hist = np.ascontiguousarray(hist, np.uint32).reshape(len(norms), -1); norms = _f32(norms); levels = _f32(levels)
    out = np.zeros(levels.size, np.float64)
    lib().orc_level_probabilities(_p(hist, C.c_uint32), hist.shape[1], _p(norms, C.c_float), norms.size, d,
                                  _p(levels, C.c_float), levels.size, _p(out, C.c_double))
    return out


def expected_code_length(p: np.ndarray, d: int):
    """(expected bits of one layer's message as the appendix writes it, expected non-zero coordinates)."""
    p = np.ascontiguousarray(p, np.float64); nz = C.c_double(0)
    bits = lib().orc_expected_code_length(_p(p, C.c_double), p.size, d, C.byref(nz))
    return float(bits), nz.value


def huffman_lengths(weights, max_len: int = 12) -> np.ndarray:
    """Code lengths of a Huffman code for the given symbol weights (every symbol gets a word)."""
    w = np.ascontiguousarray(weights, np.float64); out = np.zeros(w.size, np.uint8)
    ok = lib().orc_huffman_lengths(_p(w, C.c_double), w.size, max_len, _p(out, C.c_uint8))
    assert ok
    return out


def elias_omega(value: int) -> str:
    """Elias' recursive code word of a positive integer, as a string of '0' and '1'."""
    buf = C.create_string_buffer(160)
    n = lib().orc_elias_omega(C.c_uint64(int(value)), buf)
    return buf.value.decode()[:n]


def elias_omega_decode(bits: str):
    """(value, characters used) of the first word in `bits`; value 0 if malformed."""
    used = C.c_int(0)
    v = lib().orc_elias_omega_decode(bits.encode(), C.byref(used))
    return int(v), used.value


def canonical_codes(lengths) -> np.ndarray:
    l = np.ascontiguousarray(lengths, np.uint8); out = np.zeros(l.size, np.uint32)
    lib().orc_canonical_codes(_p(l, C.c_uint8), l.size, _p(out, C.c_uint32))
    return out


def entropy_encode_block(idx, sign, lengths, codes):
    """(words, number of bits) of one block of up to 1024 coordinates."""
    idx = np.ascontiguousarray(idx, np.uint8); sign = np.ascontiguousarray(sign, np.uint8)
    l = np.ascontiguousarray(lengths, np.uint8); c = np.ascontiguousarray(codes, np.uint32)
    words = np.zeros(1056, np.uint32)
    bits = lib().orc_entropy_encode_block(_p(idx, C.c_uint8), _p(sign, C.c_uint8), idx.size, _p(l, C.c_uint8),
                                          _p(c, C.c_uint32), _p(words, C.c_uint32))
    return words[: (bits + 31) // 32].copy(), int(bits)


def entropy_decode_block(words, count: int, lengths, codes):
    """(idx, sign, bits consumed) of one block; bits = -1 when the stream is not valid."""
    w = np.zeros(1056, np.uint32); w[: len(words)] = words
    l = np.ascontiguousarray(lengths, np.uint8); c = np.ascontiguousarray(codes, np.uint32)
    idx = np.zeros(count, np.uint8); sg = np.zeros(count, np.uint8)
    bits = lib().orc_entropy_decode_block(_p(w, C.c_uint32), count, _p(l, C.c_uint8), _p(c, C.c_uint32), l.size,
                                          _p(idx, C.c_uint8), _p(sg, C.c_uint8))
    return idx, sg, int(bits)


def alt_rates(lam: float, mu: float, qhat: float):
    """(eta, gamma) of Eq. (Alt) from the running sums lambda and mu."""
    eta = C.c_float(0); gamma = C.c_float(0)
    lib().orc_alt_rates(lam, mu, qhat, C.byref(eta), C.byref(gamma))
    return np.float32(eta.value), np.float32(gamma.value)


def sq_norm(g: np.ndarray) -> float:
    g = _f32(g)
    return float(lib().orc_sq_norm(_p(g, C.c_float), g.size))


def qoda_update_rates(gbar, X1, Y, Xhalf, X, eta, gamma) -> None:
    """As qoda_update with an extrapolation rate gamma of its own."""
    lib().orc_qoda_update_rates(_p(gbar, C.c_float), _p(X1, C.c_float), _p(Y, C.c_float), _p(Xhalf, C.c_float),
                                _p(X, C.c_float), C.c_float(float(eta)), C.c_float(float(gamma)), gbar.size)


def uniform_levels(bits: int) -> np.ndarray:
    n = 1 << bits
    return (np.arange(n, dtype=np.float64) / (n - 1)).astype(np.float32)


# --------------------------------------------------------------------- whole-message helpers
class OracleModel:
    """The K-worker pipeline on unpadded per-layer arrays: quantize -> message -> mean -> QODA.

    Mirrors Algorithm 1 of the paper for K simulated workers that share X and Y.
    """

    def __init__(self, layer_sizes: Sequence[int], bits: Sequence[int], q: int, num_workers: int,
                 seed: int):
        self.sizes = [int(s) for s in layer_sizes]
        self.bits = [int(b) for b in bits]
        self.q, self.K, self.seed = int(q), int(num_workers), int(seed)
        self.levels = [uniform_levels(b) for b in self.bits]
        self.off = np.concatenate([[0], np.cumsum(self.sizes)]).astype(np.int64)
        self.D = int(self.off[-1])
        # QODA state (Algorithm 1; initialisation V^_{k,1/2} = 0, Y_1 = 0, eta_1 = 1)
        self.X1 = None; self.Y = None; self.Xhalf = None; self.X = None
        self.S = 0.0; self.eta = np.float32(1.0); self.t = 1
        self.prev_decoded = None         # [K][D] decoded V^_{k,t-1/2}
        self.pending_sq = None
        self.norm_scope = "layer"        # "global": one norm over the worker's whole vector (Section 3.1, definition of Q)
                                         # "bucket": one norm per 128 consecutive coordinates of a layer (Section 7.1)
        self.alt_qhat = 0.0              # > 0: the alternative rates of Eq. (Alt) with this exponent
        self.lam = 0.0; self.mu = 0.0; self.gamma = np.float32(1.0)
        self.xsum = None                 # running fp64 sum of the half iterates X_{t+1/2} (ergodic average, Section 5)

    # -- ENCODE side (Algorithm 1 line 12) ------------------------------------------------
    def quantize(self, grads: np.ndarray, step: int, want_hist: bool = False):
        """grads [K][D] fp32 (unpadded, layers concatenated).  Returns a dict with the
        per-(k, layer) norms, status, idx/sign arrays, packed words, histograms, near count,
        and the per-(k, layer) squared differences to the previous decoded message."""
        K, Lr = self.K, len(self.sizes)
        norms = np.zeros((K, Lr), np.float32); status = np.zeros((K, Lr), np.int32)
        idx = np.zeros((K, self.D), np.uint8); sg = np.zeros((K, self.D), np.uint8)
        packed = [[None] * Lr for _ in range(K)]
        hist = np.zeros((K, Lr, HIST_STRIDE), np.uint32) if want_hist else None
        decoded = np.zeros((K, self.D), np.float32)
        sq = np.zeros((K, Lr), np.float64)
        near = 0
        if self.norm_scope == "bucket":
            return self._quantize_bucketed(grads, step, want_hist)
        for k in range(K):
            if self.norm_scope == "global":      # ||v||_q of the whole vector, shared by every layer of the worker
                gn, gs = layer_norm(grads[k], self.q)
            for m in range(Lr):
                a, b = int(self.off[m]), int(self.off[m + 1])
                v = grads[k, a:b]
                if self.norm_scope == "global":
                    norms[k, m], status[k, m] = gn, gs
                else:
                    norms[k, m], status[k, m] = layer_norm(v, self.q)
                i_, s_, nr = quantize_layer(v, norms[k, m], self.levels[m], self.seed, step, k, m)
                near += nr
                idx[k, a:b], sg[k, a:b] = i_, s_
                packed[k][m] = pack_layer(i_, s_, self.bits[m])
                if want_hist:
                    hist[k, m] = histogram_layer(v, norms[k, m])
                decoded[k, a:b] = decode_layer(i_, s_, norms[k, m], self.levels[m])
                prev = None if self.prev_decoded is None else self.prev_decoded[k, a:b]
                sq[k, m] = sq_diff(decoded[k, a:b], prev)
        self.pending_sq = sq
        self.cur_decoded = decoded
        return dict(norms=norms, status=status, idx=idx, sign=sg, packed=packed, hist=hist,
                    near=near, sq_diff=sq, decoded=decoded)

    def _quantize_bucketed(self, grads: np.ndarray, step: int, want_hist: bool, bucket: int = 128):
        """The quantizer applied bucket by bucket (Section 7.1: buckets of 128 coordinates): every bucket of a layer
        is a vector of its own with its own norm and the layer's level sequence; coordinate indices (the random
        numbers' counters) stay those of the layer.  A layer's histogram pools its buckets; its weight in the
        level fit is the square root of the summed squared bucket norms; status 2 if any bucket held NaN or Inf,
        else 1 if no bucket has a nonzero norm."""
        K, Lr = self.K, len(self.sizes)
        status = np.zeros((K, Lr), np.int32); weights = np.zeros((K, Lr), np.float32)
        bnorms = [[None] * Lr for _ in range(K)]
        idx = np.zeros((K, self.D), np.uint8); sg = np.zeros((K, self.D), np.uint8)
        packed = [[None] * Lr for _ in range(K)]
        hist = np.zeros((K, Lr, HIST_STRIDE), np.uint32) if want_hist else None
        decoded = np.zeros((K, self.D), np.float32)
        sq = np.zeros((K, Lr), np.float64)
        near = 0
        for k in range(K):
            for m in range(Lr):
                a, b = int(self.off[m]), int(self.off[m + 1])
                nb = (b - a + bucket - 1) // bucket
                bn = np.zeros(nb, np.float32)
                any_bad, any_live, energy = False, False, 0.0
                for i in range(nb):
                    lo, hi = a + i * bucket, min(a + (i + 1) * bucket, b)
                    v = grads[k, lo:hi]
                    bn[i], st = layer_norm(v, self.q)
                    any_bad |= st == 2; any_live |= bn[i] > 0
                    energy += float(bn[i]) * float(bn[i])
                    i_, s_, nr = quantize_layer(v, bn[i], self.levels[m], self.seed, step, k, m, first_index=lo - a)
                    near += nr
                    idx[k, lo:hi], sg[k, lo:hi] = i_, s_
                    if want_hist:
                        hist[k, m] += histogram_layer(v, bn[i])
                    decoded[k, lo:hi] = decode_layer(i_, s_, bn[i], self.levels[m])
                bnorms[k][m] = bn
                weights[k, m] = np.float32(np.sqrt(energy))
                status[k, m] = 2 if any_bad else (0 if any_live else 1)
                packed[k][m] = pack_layer(idx[k, a:b], sg[k, a:b], self.bits[m])
                prev = None if self.prev_decoded is None else self.prev_decoded[k, a:b]
                sq[k, m] = sq_diff(decoded[k, a:b], prev)
        self.pending_sq = sq
        self.cur_decoded = decoded
        return dict(norms=weights, bucket_norms=bnorms, status=status, idx=idx, sign=sg, packed=packed, hist=hist,
                    near=near, sq_diff=sq, decoded=decoded)

    def fit(self, hist: np.ndarray, norms: np.ndarray) -> None:
        """Algorithm 1 lines 2-7: refit every layer's levels from the K workers' histograms."""
        for m, d in enumerate(self.sizes):
            n = 1 << self.bits[m]
            if n < 3 or d == 0:
                continue
            new = fit_levels(hist[:, m, :], norms[:, m], d, n)
            if new is not None:
                self.levels[m] = new

    # -- DECODE + aggregate (Algorithm 1 lines 15, 17) --------------------------------------
    def mean_decoded(self, decoded: np.ndarray) -> np.ndarray:
        return aggregate(decoded)

    # -- QODA (Algorithm 1 lines 10, 17, 18 and Eq. general_stepsize) -----------------------
    def qoda_init(self, X1: np.ndarray) -> None:
        self.X1 = _f32(X1).copy(); self.Y = np.zeros_like(self.X1)
        self.Xhalf = self.X1.copy(); self.X = self.X1.copy()
        self.S = 0.0; self.eta = np.float32(1.0); self.t = 1
        self.prev_decoded = None
        self.lam = 0.0; self.mu = 0.0; self.gamma = np.float32(1.0)
        self.xsum = np.zeros(self.X1.shape, np.float64)

    def qoda_step(self) -> np.ndarray:
        """Consumes the message of the last quantize() call; returns gbar."""
        self.xsum += self.Xhalf.astype(np.float64)      # X_{t+1/2}: where this iteration's dual vectors were evaluated
        if self.alt_qhat > 0.0:
            # eta_{t+1}, gamma_{t+1} use the sums through iteration t-1; this iteration's terms come after
            self.eta, self.gamma = alt_rates(self.lam, self.mu, self.alt_qhat)
            gbar = aggregate(self.cur_decoded)
            X_old = self.X.copy()
            qoda_update_rates(gbar, self.X1, self.Y, self.Xhalf, self.X, self.eta, self.gamma)
            self.lam += sq_norm(gbar)
            self.mu += sq_diff(X_old, self.X)
            self.prev_decoded = self.cur_decoded
            self.t += 1
            return gbar
        total = 0.0
        for k in range(self.K):                       # fixed order: worker, then layer
            for m in range(len(self.sizes)):
                total += float(self.pending_sq[k, m])
        self.S, self.eta = step_size(self.S, total, self.K)
        gbar = aggregate(self.cur_decoded)
        qoda_update(gbar, self.X1, self.Y, self.Xhalf, self.X, self.eta)
        self.prev_decoded = self.cur_decoded
        self.t += 1
        return gbar
