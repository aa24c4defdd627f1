"""Pins for the oracle's record reader, expert FFN and combine (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import ftmoe_oracle as O
from paper_2608_16157_b200 import workload as W


def _bf16_bits(a: np.ndarray) -> np.ndarray:
    """float -> bf16 bit patterns via torch's round-to-nearest-even (a library routine)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def _record_bf16_by_definition(wg, wu, wd):
    """Build a record straight from the documented layout with explicit loops over (n, i)."""
    d, I = wg.shape
    rec = np.zeros(3 * I * d, dtype=np.uint16)
    gb, ub, db = _bf16_bits(wg), _bf16_bits(wu), _bf16_bits(wd)
    unit_el = 48 * d                      # 16 neurons: gate part, up part, down part of 16*d elements each
    for n in range(I):
        unit, nhalf, nrow = n // 16, (n % 16) // 8, n % 8
        for i in range(d):
            # gate / up: 1 KiB tiles of 16 neurons x 32 hidden indices: two groups of 8 rows of 64 bytes (32
            # elements); chunk (8 elements) number `chunk` of row r is stored at position chunk ^ (r >> 1)
            tile, chunk, e = i // 32, (i % 32) // 8, i % 8
            position = chunk ^ (nrow >> 1)
            at = unit * unit_el + tile * 512 + nhalf * 256 + nrow * 32 + position * 8 + e
            rec[at] = gb[i, n]
            rec[at + 16 * d] = ub[i, n]
            # down (i is the output column here): 512-byte tiles of 16 columns x the unit's 16 neurons: two
            # groups of 8 column rows of 32 bytes; the chunk of neuron half nhalf is stored at nhalf ^ (r >> 2)
            ctile, chalf, crow = i // 16, (i % 16) // 8, i % 8
            rec[unit * unit_el + 32 * d + ctile * 256 + chalf * 128 + crow * 16 + (nhalf ^ (crow >> 2)) * 8 + nrow] = db[n, i]
    return rec.view(np.uint8)


def test_unpack_bf16_record_orientation():
    d, I = 64, 32
    # all exactly representable in bf16; the periods (251, 127, 31) are coprime to every stride of the layout
    wg = ((np.arange(d * I, dtype=np.float32).reshape(d, I) % 251) - 125.0) / 4.0
    wu = -((np.arange(d * I, dtype=np.float32).reshape(d, I) % 127) - 63.0) / 8.0
    wd = (np.arange(I * d, dtype=np.float32).reshape(I, d) % 31) - 15.0
    g, u, dn = O.unpack_record(_record_bf16_by_definition(wg, wu, wd), d, I, "bf16")
    assert np.array_equal(g, wg) and np.array_equal(u, wu) and np.array_equal(dn, wd)


def _record_int4_by_definition(qg, qu, qd, sg, su, sd):
    """qX: int codes [I][d] (row = neuron); sg/su [I][d/128]; sd [I/128][d] (floats, bf16-exact).  Written section
    by section, word by word, from the documented tile order."""
    I, d = qg.shape
    G, NG, U = d // 128, I // 128, I // 16
    nwd = min(16, d // 64)
    cbw, CB = 64 * nwd, d // (64 * nwd)
    NU = (0, 0, 1, 1, 2, 2, 3, 3)                         # nibble e: neuron 4q + e//2, column g + 8*(e%2)
    out = bytearray()

    def word(nibbles):
        v = 0
        for e, c in enumerate(nibbles):
            v |= (int(c) & 0xF) << (4 * e)
        return v.to_bytes(4, "little")

    for u in range(U):                                   # section A: units of 16 neurons
        for q_ in (qg, qu):
            for grp in range(G):                          # a tile: 16 rows of 64 bytes = 4 chunks of 4 words
                for row in range(16):
                    for chunk in range(4):
                        for j in range(4):
                            i0 = 128 * grp + 32 * j + 8 * chunk
                            out += word(q_[16 * u + row, i0:i0 + 8])
        for s_ in (sg, su):
            for grp in range(G):
                for r in range(8):                        # pairs (row r, row r + 8)
                    out += _bf16_bits(np.array([s_[16 * u + r, grp], s_[16 * u + r + 8, grp]])).tobytes()
    for cb in range(CB):                                  # section B: down codes
        for ng in range(NG):
            for uu in range(8):
                for w in range(nwd):
                    for lane in range(32):
                        g, q = divmod(lane, 4)
                        for j in range(4):
                            col0 = cb * cbw + (4 * w + j) * 16
                            out += word([qd[128 * ng + 16 * uu + 4 * q + NU[e], col0 + g + 8 * (e & 1)] for e in range(8)])
    for ng in range(NG):                                  # section C: down scales
        for cb in range(CB):
            for w in range(nwd):
                for g in range(8):
                    for j in range(4):
                        col0 = cb * cbw + (4 * w + j) * 16
                        out += _bf16_bits(np.array([sd[ng, col0 + g], sd[ng, col0 + g + 8]])).tobytes()
    return np.frombuffer(bytes(out), dtype=np.uint8)


@pytest.mark.parametrize("d,I", [(256, 128), (2048, 256)])      # one / two column blocks, one / two neuron groups
def test_unpack_int4_record_by_definition(d, I):
    rng = np.random.default_rng(0)
    qg, qu, qd = (rng.integers(-8, 8, size=(I, d)) for _ in range(3))
    sg = rng.integers(1, 9, size=(I, d // 128)).astype(np.float32) / 64.0
    su = rng.integers(1, 9, size=(I, d // 128)).astype(np.float32) / 32.0
    sd = rng.integers(1, 9, size=(I // 128, d)).astype(np.float32) / 16.0
    rec = _record_int4_by_definition(qg, qu, qd, sg, su, sd)
    assert rec.size == W.LayerShape(d, I, 1, 1, "int4").expert_bytes
    wg, wu, wd = O.unpack_record(rec, d, I, "int4")
    assert np.array_equal(wg, (qg * np.repeat(sg, 128, axis=1)).T)
    assert np.array_equal(wu, (qu * np.repeat(su, 128, axis=1)).T)
    assert np.array_equal(wd, qd * np.repeat(sd, 128, axis=0))
    # all-zero codes give zero weights; code 1 with scale 1 gives column sums of x
    z = np.zeros((I, d), dtype=np.int64)
    one = np.ones((I, d), dtype=np.int64)
    s1g = np.ones((I, d // 128), dtype=np.float32)
    s1d = np.ones((I // 128, d), dtype=np.float32)
    wg0, wu0, wd0 = O.unpack_record(_record_int4_by_definition(z, z, z, s1g, s1g, s1d), d, I, "int4")
    assert not wg0.any() and not wu0.any() and not wd0.any()
    wg1, _, _ = O.unpack_record(_record_int4_by_definition(one, one, one, s1g, s1g, s1d), d, I, "int4")
    x = rng.standard_normal((3, d))
    np.testing.assert_allclose(x @ wg1, np.repeat(x.sum(axis=1, keepdims=True), I, axis=1), rtol=1e-12)


FP4_VALUES = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)     # the e2m1 magnitudes, by code & 7


def _record_mxfp4_by_definition(cg, cu, cd, bg, bu, bd):
    """cX: codes 0..15 [I][d] (row = neuron); bg/bu [I][d/32], bd [I/32][d] scale bytes.  Written section by section
    from the documented tile order."""
    I, d = cg.shape
    G, NG, U = d // 128, I // 128, I // 16
    nwd = min(16, d // 64)
    cbw, CB = 64 * nwd, d // (64 * nwd)
    out = bytearray()

    def word(nibbles):
        v = 0
        for e, c in enumerate(nibbles):
            v |= (int(c) & 0xF) << (4 * e)
        return v.to_bytes(4, "little")

    for u in range(U):
        for c_ in (cg, cu):
            for grp in range(G):
                for row in range(16):
                    for chunk in range(4):
                        for j in range(4):
                            i0 = 128 * grp + 32 * j + 8 * chunk
                            out += word(c_[16 * u + row, i0:i0 + 8])
        for b_ in (bg, bu):
            for grp in range(G):
                for r in range(8):
                    out += bytes(int(b_[16 * u + r, 4 * grp + j]) for j in range(4))
                    out += bytes(int(b_[16 * u + r + 8, 4 * grp + j]) for j in range(4))
    for cb in range(CB):
        for ng in range(NG):
            for uu in range(8):
                for w in range(nwd):
                    for lane in range(32):
                        g, q = divmod(lane, 4)
                        for j in range(4):
                            col0 = cb * cbw + (4 * w + j) * 16
                            out += word([cd[128 * ng + 16 * uu + 4 * q + e // 2, col0 + g + 8 * (e & 1)] for e in range(8)])
    for ng in range(NG):
        for cb in range(CB):
            for w in range(nwd):
                for g in range(8):
                    for j in range(4):
                        for half in range(2):
                            col = cb * cbw + (4 * w + j) * 16 + g + 8 * half
                            out += bytes(int(bd[4 * ng + m, col]) for m in range(4))
    return np.frombuffer(bytes(out), dtype=np.uint8)


@pytest.mark.parametrize("d,I", [(256, 128), (1024, 256)])
def test_unpack_mxfp4_record_by_definition(d, I):
    rng = np.random.default_rng(3)
    cg, cu, cd = (rng.integers(0, 16, size=(I, d)) for _ in range(3))
    bg = rng.integers(120, 131, size=(I, d // 32))
    bu = rng.integers(110, 127, size=(I, d // 32))
    bd = rng.integers(125, 135, size=(I // 32, d))
    rec = _record_mxfp4_by_definition(cg, cu, cd, bg, bu, bd)
    assert rec.size == W.LayerShape(d, I, 1, 1, "mxfp4").expert_bytes
    wg, wu, wd = O.unpack_record(rec, d, I, "mxfp4")
    val = np.array(FP4_VALUES)

    def deq(c, b, axis):
        return np.where(c & 8, -1.0, 1.0) * val[c & 7] * np.repeat(np.exp2(b.astype(np.float64) - 127), 32, axis=axis)

    assert np.array_equal(wg, deq(cg, bg, 1).T)
    assert np.array_equal(wu, deq(cu, bu, 1).T)
    assert np.array_equal(wd, deq(cd, bd, 0))
    # code 2 (= 1.0) everywhere with scale byte 127 (= 2**0) gives column sums of x; code 10 their negatives
    ones = np.full((I, d), 2)
    b0g, b0d = np.full((I, d // 32), 127), np.full((I // 32, d), 127)
    wg1, _, wd1 = O.unpack_record(_record_mxfp4_by_definition(ones, ones, ones | 8, b0g, b0g, b0d), d, I, "mxfp4")
    x = rng.standard_normal((3, d))
    np.testing.assert_allclose(x @ wg1, np.repeat(x.sum(axis=1, keepdims=True), I, axis=1), rtol=1e-12)
    assert np.array_equal(wd1, -np.ones((I, d)))


def _record_nvfp4_by_definition(cg, cu, cd, bg, bu, bd, scales):
    """cX: codes 0..15 [I][d] (row = neuron); bg/bu [I][d/16], bd [I/16][d] e4m3 scale bytes; scales: three floats.
    Written section by section from the documented tile order."""
    I, d = cg.shape
    G, NG, U = d // 128, I // 128, I // 16
    nwd = min(16, d // 64)
    cbw, CB = 64 * nwd, d // (64 * nwd)
    out = bytearray()

    def word(nibbles):
        v = 0
        for e, c in enumerate(nibbles):
            v |= (int(c) & 0xF) << (4 * e)
        return v.to_bytes(4, "little")

    for u in range(U):
        for c_ in (cg, cu):
            for grp in range(G):
                for row in range(16):
                    for chunk in range(4):
                        for j in range(4):
                            i0 = 128 * grp + 32 * j + 4 * chunk      # nibble e: hidden i0 + 16 (e & 1) + e // 2
                            out += word([c_[16 * u + row, i0 + 16 * (e & 1) + e // 2] for e in range(8)])
        for b_ in (bg, bu):
            for grp in range(G):
                for r in range(8):
                    out += bytes(int(b_[16 * u + r, 8 * grp + k]) for k in range(8))
                    out += bytes(int(b_[16 * u + r + 8, 8 * grp + k]) for k in range(8))
    for cb in range(CB):
        for ng in range(NG):
            for uu in range(8):
                for w in range(nwd):
                    for lane in range(32):
                        g, q = divmod(lane, 4)
                        for j in range(4):
                            col0 = cb * cbw + (4 * w + j) * 16
                            out += word([cd[128 * ng + 16 * uu + 4 * q + e // 2, col0 + g + 8 * (e & 1)] for e in range(8)])
    for ng in range(NG):
        for cb in range(CB):
            for w in range(nwd):
                for g in range(8):
                    for j in range(4):
                        for half in range(2):
                            col = cb * cbw + (4 * w + j) * 16 + g + 8 * half
                            out += bytes(int(bd[8 * ng + m, col]) for m in range(8))
    out += np.asarray(scales, dtype="<f4").tobytes()
    out += bytes(256 - 12)
    return np.frombuffer(bytes(out), dtype=np.uint8)


def test_nvfp4_block_scale_bytes_are_e4m3_numbers():
    """The reader's scale decoding against the library's float8 (e4m3) type, for every allowed byte: a record whose
    codes are all 1.0 (code 2) and whose gate scale bytes run through 0..0x7E."""
    d, I = 2048, 128                      # 128 blocks of 16 per gate row
    two = np.full((I, d), 2)
    bg = np.tile(np.arange(128) % 0x7F, (I, 1))
    bg[1] = 0x7E - np.arange(128) % 0x7F
    bu = np.full((I, d // 16), 0x38)      # 1.0
    bd = np.full((I // 16, d), 0x38)
    rec = _record_nvfp4_by_definition(two, two, two, bg, bu, bd, (1.0, 1.0, 1.0))
    wg, wu, wd = O.unpack_record(rec, d, I, "nvfp4")
    lib = torch.arange(0, 0x7F, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert lib[0x38] == 1.0 and lib[0x7E] == 448.0 and lib[0x01] == 2.0 ** -9    # the format's landmarks
    assert np.array_equal(wg[:, 0], np.repeat(lib[bg[0]], 16))
    assert np.array_equal(wg[:, 1], np.repeat(lib[bg[1]], 16))
    assert np.array_equal(wu, np.ones((d, I))) and np.array_equal(wd, np.ones((I, d)))


@pytest.mark.parametrize("d,I", [(256, 128), (1024, 256)])
def test_unpack_nvfp4_record_by_definition(d, I):
    rng = np.random.default_rng(4)
    cg, cu, cd = (rng.integers(0, 16, size=(I, d)) for _ in range(3))
    bg = rng.integers(0, 0x7F, size=(I, d // 16))
    bu = rng.integers(0x20, 0x50, size=(I, d // 16))
    bd = rng.integers(0, 0x7F, size=(I // 16, d))
    scales = (0.75, 3.0e-3, 17.0)
    rec = _record_nvfp4_by_definition(cg, cu, cd, bg, bu, bd, scales)
    assert rec.size == W.LayerShape(d, I, 1, 1, "nvfp4").expert_bytes
    wg, wu, wd = O.unpack_record(rec, d, I, "nvfp4")
    val = np.array(FP4_VALUES)
    lib = torch.arange(0, 0x7F, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()

    def deq(c, b, axis, s):
        return np.where(c & 8, -1.0, 1.0) * val[c & 7] * np.repeat(lib[b], 16, axis=axis) * float(np.float32(s))

    assert np.array_equal(wg, deq(cg, bg, 1, scales[0]).T)
    assert np.array_equal(wu, deq(cu, bu, 1, scales[1]).T)
    assert np.array_equal(wd, deq(cd, bd, 0, scales[2]))


def test_generated_nvfp4_pool_quantiser_error_bound():
    """The generator's records, read back by the oracle, against the fp32 draws.  The matrix scale maps the largest
    magnitude to 6 * 448; a block's scale byte is its amax / (6 * matrix scale) rounded to e4m3 (relative error
    <= 2**-4), so the grid step at the top of a block is at most 2 * (1 + 2**-4) * amax / 6 and every element lies
    within half of that of its draw (elements above 6 * scale after a downward rounding of the scale saturate at
    6 * scale >= amax * (1 - 2**-4))."""
    shape = W.LayerShape(d=256, inter=128, n_experts=2, top_k=1, wdtype="nvfp4")
    rec = W.make_records(shape, seed=0, layer=0, first=0, count=1)[0].numpy()
    wg, wu, wd = O.unpack_record(rec, 256, 128, "nvfp4")
    g = torch.Generator().manual_seed(W.mix64(0, 1, 0, 0))
    w = (torch.randn((3, 128, 256), generator=g) * 0.02).double().numpy()
    for got, ref, axis in ((wg.T, w[0], 1), (wu.T, w[1], 1), (wd, w[2], 0)):
        blocks = np.abs(ref).reshape((128, 16, 16) if axis == 1 else (8, 16, 256))
        amax = np.repeat(blocks.max(axis=2 if axis == 1 else 1), 16, axis=axis)
        assert np.all(np.abs(got - ref) <= amax * (1 + 2.0 ** -4) / 6 + 1e-15)
        assert np.all(np.abs(got) <= amax * (1 + 2.0 ** -4) + 1e-15)
    assert np.count_nonzero(wg) > wg.size // 2
    # finer blocks and finer scales than mxfp4: the error is smaller on the same draws
    shape_mx = W.LayerShape(d=256, inter=128, n_experts=2, top_k=1, wdtype="mxfp4")
    wg_mx = O.unpack_record(W.make_records(shape_mx, seed=0, layer=0, first=0, count=1)[0].numpy(), 256, 128, "mxfp4")[0]
    assert np.abs(wg.T - w[0]).mean() < np.abs(wg_mx.T - w[0]).mean()


def _record_mxfp4tc_by_definition(cg, cu, cd, bg, bu, bd):
    """The inputs of `_record_mxfp4_by_definition`, written as operand images block by block."""
    I, d = cg.shape
    out = bytearray()

    def image(code_of):           # code_of(r, k): r < 128 rows, k < 128 contraction indices
        for step in range(2):
            for kcore in range(2):
                for r8 in range(16):
                    for r in range(8):
                        for byte in range(16):
                            k = 64 * step + 32 * kcore + 2 * byte
                            yield (int(code_of(8 * r8 + r, k)) & 0xF) | ((int(code_of(8 * r8 + r, k + 1)) & 0xF) << 4)

    def scale_atom(scale_of):     # scale_of(r, b): b < 4 blocks of 32
        for r32 in range(32):
            for rq in range(4):
                for b in range(4):
                    yield int(scale_of(32 * rq + r32, b))

    for ng in range(I // 128):
        for st in range(d // 128):
            for c_ in (cg, cu):
                out += bytes(image(lambda r, k: c_[128 * ng + r, 128 * st + k]))
            for b_ in (bg, bu):
                out += bytes(scale_atom(lambda r, b: b_[128 * ng + r, 4 * st + b]))
    for cgp in range(d // 128):
        for st in range(I // 128):
            out += bytes(image(lambda r, k: cd[128 * st + k, 128 * cgp + r]))
            out += bytes(scale_atom(lambda r, b: bd[4 * st + b, 128 * cgp + r]))
    return np.frombuffer(bytes(out), dtype=np.uint8)


def test_unpack_mxfp4tc_record_by_definition():
    d, I = 256, 128
    rng = np.random.default_rng(5)
    cg, cu, cd = (rng.integers(0, 16, size=(I, d)) for _ in range(3))
    bg = rng.integers(120, 131, size=(I, d // 32))
    bu = rng.integers(110, 127, size=(I, d // 32))
    bd = rng.integers(125, 135, size=(I // 32, d))
    rec = _record_mxfp4tc_by_definition(cg, cu, cd, bg, bu, bd)
    assert rec.size == W.LayerShape(d, I, 1, 1, "mxfp4tc").expert_bytes
    wg, wu, wd = O.unpack_record(rec, d, I, "mxfp4tc")
    val = np.array(FP4_VALUES)

    def deq(c, b, axis):
        return np.where(c & 8, -1.0, 1.0) * val[c & 7] * np.repeat(np.exp2(b.astype(np.float64) - 127), 32, axis=axis)

    assert np.array_equal(wg, deq(cg, bg, 1).T)
    assert np.array_equal(wu, deq(cu, bu, 1).T)
    assert np.array_equal(wd, deq(cd, bd, 0))
    # the same numbers in the register-fragment order of the mxfp4 record read back identically
    wg2, wu2, wd2 = O.unpack_record(_record_mxfp4_by_definition(cg, cu, cd, bg, bu, bd), d, I, "mxfp4")
    assert np.array_equal(wg, wg2) and np.array_equal(wu, wu2) and np.array_equal(wd, wd2)


def test_generated_mxfp4tc_pool_equals_generated_mxfp4_pool():
    """Both layouts are packed from the same quantiser output: the generator's records decode to the same weights."""
    for d, I in ((256, 128), (512, 256)):
        a = W.make_records(W.LayerShape(d, I, 2, 1, "mxfp4tc"), seed=3, layer=1, first=1, count=1)[0].numpy()
        b = W.make_records(W.LayerShape(d, I, 2, 1, "mxfp4"), seed=3, layer=1, first=1, count=1)[0].numpy()
        for x, y in zip(O.unpack_record(a, d, I, "mxfp4tc"), O.unpack_record(b, d, I, "mxfp4")):
            assert np.array_equal(x, y) and np.count_nonzero(x) > x.size // 2


def test_generated_mxfp4_pool_quantiser_error_bound():
    """The generator's records, read back by the oracle, are within half a grid step of the fp32 draws: the e2m1 grid
    step is at most 2 (between 4 and 6) times the block scale 2**(floor(log2(amax)) - 2), i.e. |w - deq| <= amax / 4."""
    shape = W.LayerShape(d=256, inter=128, n_experts=2, top_k=1, wdtype="mxfp4")
    rec = W.make_records(shape, seed=0, layer=0, first=0, count=1)[0].numpy()
    wg, wu, wd = O.unpack_record(rec, 256, 128, "mxfp4")
    g = torch.Generator().manual_seed(W.mix64(0, 1, 0, 0))
    w = (torch.randn((3, 128, 256), generator=g) * 0.02).double().numpy()
    for got, ref, axis in ((wg.T, w[0], 1), (wu.T, w[1], 1), (wd, w[2], 0)):
        blocks = np.abs(ref).reshape((128, 8, 32) if axis == 1 else (4, 32, 256))
        amax = np.repeat(blocks.max(axis=2 if axis == 1 else 1), 32, axis=axis)
        assert np.all(np.abs(got - ref) <= amax / 4 + 1e-15)
        assert np.all(np.abs(got) <= 1.5 * amax + 1e-15)          # the largest element maps to 4 or 6 times the scale
    # and the records are not trivially zero
    assert np.count_nonzero(wg) > wg.size // 2


def test_generated_int4_pool_quantiser_error_bound():
    shape = W.LayerShape(d=256, inter=128, n_experts=2, top_k=1, wdtype="int4")
    rec = W.make_records(shape, seed=0, layer=0, first=0, count=1)[0].numpy()
    wg, wu, wd = O.unpack_record(rec, 256, 128, "int4")
    # regenerate the fp32 draws and check |w - deq(w)| <= scale/2 (+ bf16 rounding of the scale)
    g = torch.Generator().manual_seed(W.mix64(0, 1, 0, 0))
    w = (torch.randn((3, 128, 256), generator=g) * 0.02).double().numpy()
    for got, ref, axis in ((wg.T, w[0], 1), (wu.T, w[1], 1), (wd, w[2], 0)):
        amax = np.abs(ref).reshape((128, 2, 128) if axis == 1 else (1, 128, 256)).max(axis=2 if axis == 1 else 1)
        bound = np.repeat(amax / 7.0, 128, axis=axis) * (0.5 + 7 * 2.0 ** -8) + 1e-12
        assert np.all(np.abs(got - ref) <= bound)


def test_single_expert_is_library_swiglu_mlp():
    rng = np.random.default_rng(1)
    d, I, T = 32, 24, 5
    x = rng.standard_normal((T, d))
    wg, wu, wd = rng.standard_normal((d, I)), rng.standard_normal((d, I)), rng.standard_normal((I, d))
    xt = torch.from_numpy(x)
    ref = (torch.nn.functional.silu(xt @ torch.from_numpy(wg)) * (xt @ torch.from_numpy(wu))) @ torch.from_numpy(wd)
    np.testing.assert_allclose(O.expert_ffn(x, wg, wu, wd), ref.numpy(), rtol=1e-12, atol=1e-12)
    ids = np.zeros((T, 1), dtype=np.int32)
    w = np.ones((T, 1), dtype=np.float32)
    y = O.moe_layer(x, ids, w, lambda e: (wg, wu, wd))
    np.testing.assert_allclose(y, ref.numpy(), rtol=1e-12, atol=1e-12)


def _dense_moe(x, logits, k, experts):
    """Uncached dense MoE: every expert evaluated for every token, weighted by the masked gate."""
    T, E = logits.shape
    z = torch.from_numpy(logits).double()
    top = torch.topk(z, k, dim=1)
    gate = torch.zeros(T, E, dtype=torch.float64)
    gate.scatter_(1, top.indices, torch.softmax(top.values, dim=1))
    y = np.zeros_like(x)
    for e, (wg, wu, wd) in enumerate(experts):
        xt = torch.from_numpy(x)
        o = (torch.nn.functional.silu(xt @ torch.from_numpy(wg)) * (xt @ torch.from_numpy(wu))) @ torch.from_numpy(wd)
        y += gate[:, e:e + 1].numpy() * o.numpy()
    return y


def test_cached_layer_equals_dense_uncached_moe_for_any_slot_count():
    shape = W.LayerShape(d=256, inter=128, n_experts=8, top_k=2)
    pool = W.make_records(shape, seed=0, layer=0, first=0, count=8).numpy()
    experts = [O.unpack_record(pool[e], 256, 128, "bf16") for e in range(8)]
    cm = O.CostModel(shape.expert_bytes, 50000, 0, 50000, 6000000)
    ys = {}
    for n_slots in (0, 4, 8):
        layer = O.OracleLayer(256, 128, 8, 2, n_slots, "bf16", pool, cm)
        out = []
        for step in range(3):
            logits = W.normal_logits(8, 8, 0, step)      # continuous: no ties, torch.topk agrees
            xb = W.noise_x(8, 256, 0, step, 0).view(torch.int16).numpy().view(np.uint16)
            r = layer.step(logits, xb)
            ref = _dense_moe(O.bf16_to_f64(xb), logits, 2, experts)
            np.testing.assert_allclose(r.y, ref, rtol=1e-6, atol=1e-8)   # gate weights are rounded to fp32
            out.append(r.y)
        ys[n_slots] = out
    for step in range(3):
        assert np.array_equal(ys[0][step], ys[4][step]) and np.array_equal(ys[4][step], ys[8][step])


def test_algebraic_properties_of_the_layer():
    rng = np.random.default_rng(2)
    d, I, E, k, T = 16, 12, 5, 3, 7
    x = rng.standard_normal((T, d))
    logits = rng.standard_normal((T, E)).astype(np.float32)
    ids, w = O.route(logits, k)
    same = (rng.standard_normal((d, I)), rng.standard_normal((d, I)), rng.standard_normal((I, d)))
    # identical experts: the gate weights sum to one, so y = FFN(x)
    y = O.moe_layer(x, ids, w, lambda e: same)
    np.testing.assert_allclose(y, O.expert_ffn(x, *same), rtol=1e-6, atol=1e-6)
    # W_down = 0 -> 0 ; scaling W_down scales y
    experts = [(rng.standard_normal((d, I)), rng.standard_normal((d, I)), rng.standard_normal((I, d))) for _ in range(E)]
    y0 = O.moe_layer(x, ids, w, lambda e: (experts[e][0], experts[e][1], 0 * experts[e][2]))
    assert not y0.any()
    y1 = O.moe_layer(x, ids, w, lambda e: experts[e])
    y3 = O.moe_layer(x, ids, w, lambda e: (experts[e][0], experts[e][1], 3.0 * experts[e][2]))
    np.testing.assert_allclose(y3, 3.0 * y1, rtol=1e-12)
    # a shared expert adds its FFN with weight one
    ys = O.moe_layer(x, ids, w, lambda e: experts[e], shared=[same])
    np.testing.assert_allclose(ys - y1, O.expert_ffn(x, *same), rtol=1e-9, atol=1e-9)
