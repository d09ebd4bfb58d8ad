"""Pins for the oracle's bit packing and storage formulas (no GPU)."""
import itertools
import os

import numpy as np
import pytest

from paper_2605_24058_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_written_words_role_a(oracle):
    # one row of 64 columns: +1 at columns 0, 1, 31, 32, 63, -1 elsewhere
    s = -np.ones((1, 64), np.int8)
    for c in (0, 1, 31, 32, 63):
        s[0, c] = 1
    got = oracle.pack_signs(s, 0)
    assert got.tolist() == [0x80000003, 0x80000001]
    # two rows of 40 columns: one 64-column block, one 64-bit group per row, pad bits stay 0
    s = -np.ones((2, 40), np.int8)
    s[0, 39] = 1
    s[1, 0] = 1
    s[1, 33] = 1
    got = oracle.pack_signs(s, 0)
    assert got.tolist() == [0x0, 0x80, 0x1, 0x2]
    # two rows of 70 columns: block 0 = (row 0, row 1), block 1 = (row 0, row 1)
    s = -np.ones((2, 70), np.int8)
    s[0, 1] = 1       # block 0, row 0, low word bit 1
    s[1, 63] = 1      # block 0, row 1, high word bit 31
    s[0, 64] = 1      # block 1, row 0, low word bit 0
    s[1, 69] = 1      # block 1, row 1, low word bit 5
    got = oracle.pack_signs(s, 0)
    assert got.tolist() == [0x2, 0x0, 0x0, 0x80000000, 0x1, 0x0, 0x20, 0x0]


def test_hand_written_words_role_b(oracle):
    # d_out=5, r=8: dense stream, bit j*8+k; 40 bits -> 2 words
    s = -np.ones((5, 8), np.int8)
    s[0, 0] = 1      # bit 0
    s[1, 7] = 1      # bit 15
    s[3, 7] = 1      # bit 31
    s[4, 0] = 1      # bit 32 -> word 1 bit 0
    s[4, 7] = 1      # bit 39 -> word 1 bit 7
    got = oracle.pack_signs(s, 1)
    assert got.tolist() == [0x80008001, 0x81]
    # r=16: one 16-bit group per output channel, two channels per word
    s = -np.ones((2, 16), np.int8)
    s[0, 15] = 1
    s[1, 0] = 1
    assert oracle.pack_signs(s, 1).tolist() == [0x00018000]


def test_zero_counts_as_plus_one(oracle):
    s = np.array([[0, -1, 5, -128]], dtype=np.int8)
    assert oracle.pack_signs(s, 0).tolist() == [0b0101, 0]
    assert oracle.unpack_signs(np.array([0b0101, 0], np.uint32), 1, 4, 0).tolist() == [[1, -1, 1, -1]]


@pytest.mark.parametrize("role", [0, 1])
def test_exhaustive_round_trip_tiny(oracle, role):
    rows, cols = (2, 5) if role == 0 else (5, 2)
    for bits in itertools.product((-1, 1), repeat=rows * cols):
        s = np.array(bits, np.int8).reshape(rows, cols)
        p = oracle.pack_signs(s, role)
        assert np.array_equal(oracle.unpack_signs(p, rows, cols, role), s)
        assert sum(bin(int(w)).count("1") for w in p) == int((s == 1).sum())


@pytest.mark.parametrize("rows,cols,role", [(16, 4096, 0), (8, 250, 0), (3, 33, 0), (64, 11008, 0),
                                            (4096, 16, 1), (250, 8, 1), (33, 3, 1), (11008, 64, 1),
                                            (7, 5, 1)])
def test_random_round_trip_popcount_and_size(oracle, rows, cols, role):
    rng = np.random.default_rng(rows * 131 + cols)
    s = rng.integers(0, 2, size=(rows, cols)).astype(np.int8) * 2 - 1
    p = oracle.pack_signs(s, role)
    n_words = ((cols + 63) // 64) * rows * 2 if role == 0 else (rows * cols + 31) // 32
    assert p.size == n_words == oracle.packed_words(rows, cols, role)
    assert np.array_equal(oracle.unpack_signs(p, rows, cols, role), s)
    pop = int(np.unpackbits(p.view(np.uint8)).sum())
    assert pop == int((s == 1).sum())          # so every pad bit is 0
    # independent statement of the layout with numpy bit ops
    if role == 0:
        nb = (cols + 63) // 64
        padded = np.zeros((rows, nb * 64), np.uint8)
        padded[:, :cols] = (s == 1)
        blocks = padded.reshape(rows, nb, 64).transpose(1, 0, 2)          # block-major, then row
        want = np.packbits(np.ascontiguousarray(blocks), axis=2, bitorder="little").view(np.uint32).reshape(-1)
    else:
        flat = np.zeros(n_words * 32, np.uint8)
        flat[:rows * cols] = (s == 1).reshape(-1)
        want = np.packbits(flat, bitorder="little").view(np.uint32)
    assert np.array_equal(p, want)


def test_carrier_footprint_is_one_bit_per_sign(oracle):
    for d_in, d_out, r in [(4096, 4096, 16), (4096, 11008, 16), (11008, 4096, 64), (256, 256, 8)]:
        words = oracle.packed_words(r, d_in, 0) + oracle.packed_words(d_out, r, 1)
        assert words * 32 == r * (d_in + d_out)


def _llama_shapes():
    return [(di, do) for _ in range(workloads.N_LAYERS) for (_, di, do) in workloads.LAYER_PROJECTIONS]


def test_sizes_the_paper_prints(oracle):
    shapes = _llama_shapes()
    assert len(shapes) == 224
    with open(os.path.join(GOLDEN, "paper_sizes.txt")) as f:
        rows = [ln.split(None, 5) for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 8
    for kind, rank, ell, printed, tol, where in rows:
        rank, ell, printed, tol = int(rank), int(ell), float(printed), float(tol)
        if kind == "lora_fp16":
            bits = sum(oracle.lora_fp16_bits(di, do, rank) for di, do in shapes)
        else:
            bits = sum(oracle.adapter_bits(di, do, rank, ell) for di, do in shapes)
        mib = bits / 8 / 2 ** 20
        assert abs(mib - printed) <= tol, (kind, rank, mib, printed, where)


def test_bits_formula_by_hand(oracle):
    # Eq. 5 on numbers small enough to check by eye: R(N+M) + 16 l (N+R+M)
    assert oracle.adapter_bits(3, 5, 2, 1) == 2 * 8 + 16 * 10
    assert oracle.adapter_bits(3, 5, 2, 3) == 2 * 8 + 48 * 10
    assert oracle.adapter_bits(4096, 4096, 16, 1) == 16 * 8192 + 16 * (8192 + 16)
    assert oracle.lora_fp16_bits(4096, 11008, 16) == 16 * 16 * 15104


def test_bandwidth_ratio_and_bpw(oracle):
    with open(os.path.join(GOLDEN, "paper_ratios.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for r0, printed, tol in rows:
        assert abs(oracle.bandwidth_ratio(4096, 4096, int(r0)) - float(printed)) <= float(tol)
    # the ratio tends to 16 and BPW_tot to 1 as r0, N, M grow (Eq. 6 and the Analysis paragraph)
    assert abs(oracle.bandwidth_ratio(2 ** 22, 2 ** 22, 2 ** 16) - 16.0) < 0.01
    assert abs(oracle.bpw_tot(2 ** 22, 2 ** 22, 2 ** 16, 1, 2 ** 16) - 1.0) < 1e-3
    # BPW_tot = BPW_bc + 16 l (N+R+M) / (r0 (N+M))
    got = oracle.bpw_tot(4096, 11008, 32, 2, 16)
    want = 32 / 16 + 16 * 2 * (4096 + 32 + 11008) / (16 * (4096 + 11008))
    assert abs(got - want) < 1e-12


def test_workload_generator_is_seeded_and_shaped():
    p = workloads.config0()
    q = workloads.config0()
    assert p.x.dtype == np.float32 and p.x.shape == (64, 256) and p.A_sign.shape == (8, 256)
    assert np.array_equal(p.x, q.x) and np.array_equal(p.B_sign, q.B_sign)
    assert set(np.unique(p.A_sign)) == {-1, 1}
    b = workloads.make_projection(64, 32, 8, 4, "bf16", seed=1, outlier_frac=0.05)
    assert b.x.dtype == np.uint16 and b.x_f64().shape == (4, 64)
    # bf16 rounding is round-to-nearest-even
    vals = np.array([1.0, 1.00390625, 1.01171875, -3.0e38], np.float32)   # ties at 1+2^-8, 1+3*2^-8
    bits = workloads.to_bf16_bits(vals)
    assert bits.tolist()[:3] == [0x3F80, 0x3F80, 0x3F82]
    assert workloads.algorithmic_bytes(2048, 4096, 4096, 16, 2) == 50380864
