"""Glue between the CUDA plan's padded layout and the oracle's per-layer arrays (tests only)."""
import numpy as np
import torch


def to_unpadded(plan, t: torch.Tensor) -> np.ndarray:
    """[K][D_pad] (or [D_pad]) device tensor -> [K][D] (or [D]) numpy array, layers concatenated."""
    a = t.detach().cpu().numpy()
    one = a.ndim == 1
    if one:
        a = a[None, :]
    parts = [a[:, o:o + d] for o, d in zip(plan.elem_offsets, plan.layer_sizes)]
    out = np.concatenate(parts, axis=1) if parts else np.zeros((a.shape[0], 0), a.dtype)
    return out[0] if one else out


def to_padded(plan, a: np.ndarray, device="cuda") -> torch.Tensor:
    """Inverse of to_unpadded (padding = 0)."""
    one = a.ndim == 1
    if one:
        a = a[None, :]
    out = np.zeros((a.shape[0], plan.padded_elems), a.dtype)
    off = 0
    for o, d in zip(plan.elem_offsets, plan.layer_sizes):
        out[:, o:o + d] = a[:, off:off + d]; off += d
    t = torch.from_numpy(out).to(device)
    return t[0].contiguous() if one else t


def oracle_model(orc, plan):
    m = orc.OracleModel(plan.layer_sizes, plan.bits, plan.q, plan.num_workers, plan.seed)
    for i in range(plan.num_layers):
        m.levels[i] = np.array(plan.lq_get_levels(i), np.float32)
    return m


def compare_messages(orc, plan, packed_gpu: torch.Tensor, ref: dict):
    """Word-exact comparison of the GPU message with the oracle's.  Returns (number of
    coordinates whose sign or index differs, number of words that differ outside those)."""
    pk = packed_gpu.detach().cpu().numpy().view(np.uint32)
    bad_coords = 0; stray_words = 0
    off = np.concatenate([[0], np.cumsum(plan.layer_sizes)]).astype(np.int64)
    for k in range(plan.num_workers):
        for m, (d, b) in enumerate(zip(plan.layer_sizes, plan.bits)):
            nw = orc.packed_words(d, b)
            got = pk[k, plan.word_offsets[m]: plan.word_offsets[m] + nw]
            want = ref["packed"][k][m]
            if np.array_equal(got, want):
                continue
            gi, gs = orc.unpack_layer(got, d, b)
            a, e = int(off[m]), int(off[m + 1])
            diff = (gi != ref["idx"][k, a:e]) | (gs != ref["sign"][k, a:e])
            bad_coords += int(diff.sum())
            # words that differ although all real coordinates agree = layout / padding error
            if not diff.any():
                stray_words += int((got != want).sum())
    return bad_coords, stray_words


def bucket_norms_by_layer(plan, nm: torch.Tensor):
    """Bucket scope: the [K][8 * blocks] norms buffer -> per layer an array [K][ceil(d / 128)], plus the largest
    absolute value found in the slots of rows past the layers' ends (must be 0)."""
    a = nm.detach().cpu().numpy()
    out, stray, block_off = [], 0.0, 0
    for d in plan.layer_sizes:
        nblocks = (d + 1023) // 1024
        nb = (d + 127) // 128
        seg = a[:, 8 * block_off: 8 * (block_off + nblocks)]
        out.append(seg[:, :nb].copy())
        if seg[:, nb:].size:
            stray = max(stray, float(np.abs(seg[:, nb:]).max()))
        block_off += nblocks
    return out, stray
