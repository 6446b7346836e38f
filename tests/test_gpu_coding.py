"""GPU parity of the entropy stage (Huffman code on the level symbols) through the C ABI: stream words and
block offsets against the oracle's encoder block by block, the round trip back to the fixed-width message, the
size of a fitted code against the entropy bounds, and the handling of short buffers and broken streams."""
import math

import numpy as np
import pytest
import torch

from helpers import oracle_model, to_unpadded

pytestmark = pytest.mark.gpu
SEED = 0x5EED0DA


@pytest.fixture(scope="module")
def lqm():
    import paper_2505_14371_b200 as pkg
    pkg.load_library()
    return pkg


def _message(lqm, sizes, bits, K, seed, dist_scale=0.05):
    plan = lqm.Plan(sizes, bits, 2, K, SEED + seed)
    g = torch.Generator(device="cuda").manual_seed(seed)
    grads = torch.randn((K, plan.padded_elems), generator=g, device="cuda") ** 3 * dist_scale
    packed = plan.empty_packed(); norms = plan.empty_norms(); hist = plan.zero_hist()
    plan.lq_quantize_pack(grads, 1, packed, norms, hist=hist)
    return plan, grads, packed, norms, hist


def _canonical(orc, plan, packed):
    """The message with the sign bit cleared wherever the level index is 0 (the stream carries no sign there)."""
    pk = packed.cpu().numpy().view(np.uint32).copy()
    for k in range(plan.num_workers):
        for m, (d, b) in enumerate(zip(plan.layer_sizes, plan.bits)):
            nw = orc.packed_words(d, b)
            sl = slice(plan.word_offsets[m], plan.word_offsets[m] + nw)
            idx, sg = orc.unpack_layer(pk[k, sl], d, b)
            pk[k, sl] = orc.pack_layer(idx, sg * (idx != 0), b)
    return pk


def _encode(plan, packed, capacity=None):
    cap = plan.lq_plan_blocks() * 416 if capacity is None else capacity       # 1024 coordinates x 13 bits at most per block
    stream = torch.full((plan.num_workers, max(cap, 1)), -1, dtype=torch.int32, device="cuda")
    offs = torch.zeros((plan.num_workers, plan.lq_plan_blocks() + 1), dtype=torch.int32, device="cuda")
    plan.lq_entropy_encode(packed, stream, offs)
    torch.cuda.synchronize()
    return stream, offs


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 8])
def test_stream_matches_the_oracle_and_round_trips(lqm, orc, bits):
    sizes = [0, 1, 33, 1023, 1024, 1025, 5000, 3, 20000]
    plan, grads, packed, norms, hist = _message(lqm, sizes, bits, 2, bits)
    n = 1 << bits
    rng = np.random.default_rng(bits)
    lengths = {}
    for m in range(plan.num_layers):
        if m % 4 == 2 and bits <= 5:                                  # the universal recursive code where it fits
            lengths[m] = lqm.lq_code_universal(n)
            plan.lq_code_set(m, lengths[m])
        elif m % 2 == 0:                                              # a Huffman code on some layers, the flat code on others
            lengths[m] = lqm.lq_code_build(rng.dirichlet(np.ones(n) * 0.3))
            plan.lq_code_set(m, lengths[m])
        else:
            lengths[m] = [bits] * n
        assert plan.lq_code_get(m) == lengths[m]
    stream, offs = _encode(plan, packed)
    model = oracle_model(orc, plan)
    ref = model.quantize(to_unpadded(plan, grads), 1)
    S = stream.cpu().numpy().view(np.uint32); O = offs.cpu().numpy().astype(np.int64)
    off = np.concatenate([[0], np.cumsum(sizes)])
    for k in range(plan.num_workers):
        g = 0; pos = 0
        for m, d in enumerate(sizes):
            l = np.uint8(lengths[m]); c = orc.canonical_codes(l)
            for blk in range((d + 1023) // 1024):
                lo = off[m] + blk * 1024; hi = min(off[m] + d, lo + 1024)
                words, nbits = orc.entropy_encode_block(ref["idx"][k, lo:hi], ref["sign"][k, lo:hi], l, c)
                assert O[k, g] == pos, (k, m, blk)
                assert np.array_equal(S[k, pos: pos + words.size], words), (k, m, blk)
                pos += words.size; g += 1
        assert g == plan.lq_plan_blocks() and O[k, g] == pos
    back = torch.full_like(packed, -1)
    plan.lq_entropy_decode(stream, offs, back)
    torch.cuda.synchronize()
    assert plan.lq_entropy_status() == 0
    assert np.array_equal(back.cpu().numpy().view(np.uint32), _canonical(orc, plan, packed))
    # the run offsets (side data for the parallel decoder): for run r of a block, the bits of the coordinates that
    # precede it in the block's stream order s = 32 lane + p, from the definition; the stream itself is unchanged
    runs = plan.empty_run_offsets()
    stream2 = torch.full_like(stream, -1); offs2 = torch.zeros_like(offs)
    plan.lq_entropy_encode(packed, stream2, offs2, runs)
    torch.cuda.synchronize()
    assert torch.equal(offs, offs2)
    R = runs.cpu().numpy().view(np.uint16)
    for k in range(plan.num_workers):
        assert np.array_equal(stream2[k, : O[k, -1]].cpu().numpy(), stream[k, : O[k, -1]].cpu().numpy())
        g = 0
        for m, d in enumerate(sizes):
            l = np.array(lengths[m], np.int64)
            for blk in range((d + 1023) // 1024):
                ss = np.arange(1024); lane, pp = ss // 32, ss % 32
                coord = blk * 1024 + 128 * (pp // 4) + 4 * lane + pp % 4          # coordinate of stream position s
                real = coord < d
                ix = np.zeros(1024, np.int64); ix[real] = ref["idx"][k, off[m] + coord[real]]
                nbits = np.where(real, l[ix] + (ix != 0), 0)
                want = np.concatenate([[0], np.cumsum(nbits)])[0:1024:128]
                assert np.array_equal(R[k, g].astype(np.int64), want), (k, m, blk)
                g += 1
    back2 = torch.full_like(packed, -1)
    plan.lq_entropy_decode(stream, offs, back2, runs)
    torch.cuda.synchronize()
    assert plan.lq_entropy_status() == 0
    assert torch.equal(back2, back)
    # offsets that do not belong to the stream are reported, never followed out of bounds
    bad_runs = runs.clone(); bad_runs[:, :, 3] += 1
    plan.lq_entropy_decode(stream, offs, back2, bad_runs)
    torch.cuda.synchronize()
    if plan.lq_plan_blocks() > 0:
        assert plan.lq_entropy_status() != 0
    wild = torch.full_like(runs, 32767)
    plan.lq_entropy_decode(stream, offs, back2, wild)
    torch.cuda.synchronize()
    assert plan.lq_entropy_status() != 0 and plan.lq_entropy_status() == 0
    # what the decoder rebuilds decodes to the same values
    g1 = torch.empty(plan.padded_elems, device="cuda"); g2 = torch.empty_like(g1)
    plan.lq_decode_aggregate(packed, norms, g1); plan.lq_decode_aggregate(back, norms, g2)
    assert np.array_equal(to_unpadded(plan, g1), to_unpadded(plan, g2))              # padding between layers aside


@pytest.mark.parametrize("code", ["zero_is_one_bit", "flat", "zero_is_long"])
def test_untouched_rows_and_blocks(lqm, orc, code):
    """Messages with untouched rows, untouched blocks and an untouched layer end, under three codes: level 0 sent as
    the one-bit word "0" (what a fitted code gives it: runs of zero bits, which neither side walks), the flat code
    (level 0 is b zero bits), and a code whose word for level 0 is long and not all zeros (nothing can be left out).
    Stream and run offsets against the oracle's encoder block by block, and the round trip with and without the offsets."""
    bits, K = 3, 2
    sizes = [7 * 1024 + 300, 4 * 1024, 2048 + 128 * 3 + 5]
    plan = lqm.Plan(sizes, [bits] * 3, 2, K, SEED + 77)
    g = torch.Generator(device="cuda").manual_seed(77)
    grads = torch.randn((K, plan.padded_elems), generator=g, device="cuda") ** 3 * 0.05
    for k in range(K):
        for m in range(3):
            v = grads[k, plan.elem_offsets[m]: plan.elem_offsets[m] + sizes[m]]
            rows = torch.rand((sizes[m] + 127) // 128, generator=g, device="cuda") < 0.75       # untouched rows of 128
            v[rows.repeat_interleave(128)[: sizes[m]]] = 0
        grads[k, plan.elem_offsets[0] + 2048: plan.elem_offsets[0] + 4096] = 0                  # two untouched blocks
        grads[k, plan.elem_offsets[1]: plan.elem_offsets[1] + 1024 * (1 + k)] = 0
        grads[k, plan.elem_offsets[2] + 2048: plan.elem_offsets[2] + sizes[2]] = 0              # an untouched partial block
    packed = plan.empty_packed(); norms = plan.empty_norms()
    plan.lq_quantize_pack(grads, 1, packed, norms)
    n = 1 << bits
    weights = {"zero_is_one_bit": [0.9] + [0.1 / (n - 1)] * (n - 1), "zero_is_long": [0.001, 0.5, 0.25, 0.12, 0.06, 0.03, 0.02, 0.019]}
    lengths = [bits] * n if code == "flat" else lqm.lq_code_build(weights[code])
    if code == "zero_is_one_bit":
        assert lengths[0] == 1
    if code == "zero_is_long":
        assert lengths[0] > 3
    for m in range(3):
        plan.lq_code_set(m, lengths)
    runs = plan.empty_run_offsets()
    cap = plan.lq_plan_blocks() * 416
    stream = torch.full((K, cap), -1, dtype=torch.int32, device="cuda")
    offs = torch.zeros((K, plan.lq_plan_blocks() + 1), dtype=torch.int32, device="cuda")
    plan.lq_entropy_encode(packed, stream, offs, runs)
    torch.cuda.synchronize()
    model = oracle_model(orc, plan)
    ref = model.quantize(to_unpadded(plan, grads), 1)
    S = stream.cpu().numpy().view(np.uint32); O = offs.cpu().numpy().astype(np.int64); R = runs.cpu().numpy().view(np.uint16)
    off = np.concatenate([[0], np.cumsum(sizes)])
    l = np.uint8(lengths); c = orc.canonical_codes(l); l64 = l.astype(np.int64)
    for k in range(K):
        gb = 0; pos = 0
        for m, d in enumerate(sizes):
            for blk in range((d + 1023) // 1024):
                lo = off[m] + blk * 1024; hi = min(off[m] + d, lo + 1024)
                words, _ = orc.entropy_encode_block(ref["idx"][k, lo:hi], ref["sign"][k, lo:hi], l, c)
                assert O[k, gb] == pos and np.array_equal(S[k, pos: pos + words.size], words), (k, m, blk)
                ss = np.arange(1024); lane, pp = ss // 32, ss % 32
                coord = blk * 1024 + 128 * (pp // 4) + 4 * lane + pp % 4
                real = coord < d
                ix = np.zeros(1024, np.int64); ix[real] = ref["idx"][k, off[m] + coord[real]]
                nb = np.where(real, l64[ix] + (ix != 0), 0)
                assert np.array_equal(R[k, gb].astype(np.int64), np.concatenate([[0], np.cumsum(nb)])[0:1024:128]), (k, m, blk)
                pos += words.size; gb += 1
        assert O[k, gb] == pos
    want = _canonical(orc, plan, packed)
    for r in (runs, None):
        back = torch.full_like(packed, -1)
        plan.lq_entropy_decode(stream, offs, back, r)
        torch.cuda.synchronize()
        assert plan.lq_entropy_status() == 0
        assert np.array_equal(back.cpu().numpy().view(np.uint32), want)
    # a one in the middle of a run of zero bits is a different message, not an untouched row: with the one-bit word for
    # level 0 the decoder must not take the run for zeros
    if code == "zero_is_one_bit":
        k, gb = 0, 2                                                     # an untouched block of worker 0
        first = int(O[k, gb])
        assert np.all(S[k, first: int(O[k, gb + 1])] == 0)
        broken = stream.clone(); broken[k, first + 1] = 1 << 7
        back = torch.full_like(packed, -1)
        plan.lq_entropy_decode(broken, offs, back, runs)
        torch.cuda.synchronize()
        got = back.cpu().numpy().view(np.uint32)
        assert plan.lq_entropy_status() != 0 or not np.array_equal(got, want)


def test_fitted_code_beats_the_fixed_width_and_meets_the_entropy_bound(lqm, orc):
    """Codes built from the estimated level probabilities: the stream is shorter than the fixed-width message, and the
    bits spent on level words per coordinate lie between the empirical entropy and the entropy + 1."""
    sizes = [200000, 50000]
    plan, grads, packed, norms, hist = _message(lqm, sizes, 4, 3, 99)
    K = plan.num_workers
    plan.lq_fit_levels(hist, norms, K)
    hist.zero_()
    plan.lq_quantize_pack(grads, 2, packed, norms, hist=hist)                    # fitted levels
    probs = torch.zeros((plan.num_layers, 256), dtype=torch.float64, device="cuda")
    counts = torch.zeros((K, plan.num_layers, 256), dtype=torch.int32, device="cuda")
    plan.lq_level_probabilities(hist, norms, K, probs)
    plan.lq_symbol_counts(packed, counts)
    P = probs.cpu().numpy(); Cn = counts.cpu().numpy().astype(np.float64)
    for m in range(plan.num_layers):
        plan.lq_code_set(m, lqm.lq_code_build(P[m, :16]))
    stream, offs = _encode(plan, packed)
    O = offs.cpu().numpy().astype(np.int64)
    assert np.all(O[:, -1] < 0.9 * plan.packed_words)                              # at least 10 % shorter than 5 bits / coordinate
    total_bits = 0.0; bound_lo = 0.0; bound_hi = 0.0
    for m, d in enumerate(sizes):
        l = np.array(plan.lq_code_get(m), np.float64)
        for k in range(K):
            f = Cn[k, m, :16] / d
            H = -sum(x * math.log2(x) for x in f if x > 0)
            spent = float((f * l).sum())                                           # level-word bits per coordinate
            assert H - 1e-9 <= spent <= H + 1.0 + 0.05                            # code from the estimate, not from f itself
            total_bits += d * (spent + (1.0 - f[0]))
    assert abs(O[:, -1].sum() * 32 - total_bits) <= 32 * K * plan.lq_plan_blocks()   # block padding to whole words
    back = torch.empty_like(packed)
    plan.lq_entropy_decode(stream, offs, back)
    assert plan.lq_entropy_status() == 0
    assert np.array_equal(back.cpu().numpy().view(np.uint32), _canonical(orc, plan, packed))


def test_short_buffer_and_broken_stream_are_reported_not_faulted(lqm):
    sizes = [9000, 100]
    plan, grads, packed, norms, hist = _message(lqm, sizes, 3, 2, 5)
    full_stream, full_offs = _encode(plan, packed)
    need = int(full_offs[:, -1].max())
    stream, offs = _encode(plan, packed, capacity=need // 2)                       # too small: offsets still complete
    assert torch.equal(offs, full_offs) and int(offs[:, -1].max()) > stream.shape[1]
    first_half = full_stream[:, : need // 2]
    fits = offs[0, 1:] <= need // 2                                                 # blocks that fit were written
    last_fit = int(offs[0][1:][fits].max())
    assert torch.equal(stream[0, :last_fit], first_half[0, :last_fit])
    with pytest.raises(lqm.LqError):
        plan.lq_code_set(0, [1, 1, 2, 3, 3, 3, 3, 3])                               # violates Kraft's inequality
    with pytest.raises(lqm.LqError):
        plan.lq_code_set(0, [3] * 7)                                                # wrong alphabet size
    # an incomplete code (Kraft sum < 1) leaves bit patterns without a word: a stream of ones then decodes to nothing
    plan.lq_code_set(0, [2, 2, 3, 3, 4, 4, 4, 5])
    ones = torch.full_like(full_stream, -1)
    back = torch.empty_like(packed)
    plan.lq_entropy_decode(ones, full_offs, back)
    assert plan.lq_entropy_status() != 0 and plan.lq_entropy_status() == 0         # reported once, then cleared
