"""GPU parity: the CUDA path through the C ABI against the float64 oracle,
element by element on the same seeded inputs."""
import functools

import numpy as np
import pytest
import torch

from paper_2605_24058_b200 import lordba, workloads
from gpu_util import DeviceProj, assert_close, np_to_torch, oracle_forward, torch_to_f64

pytestmark = pytest.mark.gpu

# "auto" is what a caller gets (the register-streaming kernel where the shape allows it, else
# the FMA kernel); "tc" pins the tcgen05/TMA kernel and skips the shapes it does not take.
VARIANTS = [("fma", lordba.VARIANT_FMA), ("tc", lordba.VARIANT_TC), ("auto", lordba.VARIANT_AUTO)]


@pytest.fixture(autouse=True)
def _reset_variant():
    lordba.set_variant(lordba.VARIANT_AUTO)
    yield
    lordba.set_variant(lordba.VARIANT_AUTO)
    assert lordba.device_status() == 0


def skip_unsupported(fn):
    """A pinned kernel family answers LORDBA_EUNSUPPORTED for shapes it does not take: skip those."""
    @functools.wraps(fn)
    def wrapper(*args, **kwargs):
        try:
            return fn(*args, **kwargs)
        except lordba.LordbaError as e:
            if e.status == 2 and lordba.get_variant() != lordba.VARIANT_AUTO:
                pytest.skip("shape not supported by the pinned kernel family")
            raise
    return wrapper


# ---------------------------------------------------------------- packing: bit-exact

@pytest.mark.parametrize("rows,cols,role", [(8, 256, 0), (16, 4096, 0), (64, 11008, 0), (3, 33, 0),
                                            (5, 1000, 0), (1, 1, 0),
                                            (256, 8, 1), (4096, 16, 1), (11008, 64, 1), (33, 3, 1),
                                            (1000, 5, 1), (1, 1, 1), (11008, 16, 1)])
def test_pack_unpack_bit_exact(oracle, rows, cols, role):
    rng = np.random.default_rng(rows * 7 + cols + role)
    s = (rng.integers(0, 2, size=(rows, cols)) * 2 - 1).astype(np.int8)
    s_dev = torch.from_numpy(s).cuda()
    packed = lordba.pack_signs(s_dev, role)
    want = oracle.pack_signs(s, role)
    got = packed.cpu().numpy().view(np.uint32)
    assert got.shape == want.shape and np.array_equal(got, want)
    back = lordba.unpack_signs(packed, rows, cols, role).cpu().numpy()
    assert np.array_equal(back, s)
    assert np.array_equal(back, oracle.unpack_signs(want, rows, cols, role))


def test_pack_sign_of_zero_and_odd_values(oracle):
    s = np.array([[0, -1, 5, -128, 127, 0, -2, 1] * 9], dtype=np.int8)      # 72 columns
    for role in (0, 1):
        got = lordba.pack_signs(torch.from_numpy(s).cuda(), role).cpu().numpy().view(np.uint32)
        assert np.array_equal(got, oracle.pack_signs(s, role))


def test_pack_overwrites_stale_words(oracle):
    s = -np.ones((2, 40), np.int8)
    dev = torch.from_numpy(s).cuda()
    out = lordba.pack_signs(dev, 0)
    assert out.cpu().numpy().view(np.uint32).tolist() == [0, 0, 0, 0]


# ---------------------------------------------------------------- forward: the five configs

@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_config0_tiny_fp32(oracle, vname, variant):
    lordba.set_variant(variant)
    p = workloads.config0()
    d = DeviceProj(p)
    d.forward()
    assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "f32", "config0/" + vname)


@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_config1_attention_full_size(oracle, vname, variant):
    lordba.set_variant(variant)
    p = workloads.config1()
    d = DeviceProj(p)
    d.forward()
    assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "config1/" + vname)


@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_config2_mlp_full_size(oracle, vname, variant):
    lordba.set_variant(variant)
    for p in workloads.config2():
        d = DeviceProj(p)
        d.forward()
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "config2/%s/%s" % (p.name, vname))
        del d


@pytest.mark.parametrize("T", [1, 8, 32, 64])
@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_config3_decode_layer_batched(oracle, T, vname, variant):
    lordba.set_variant(variant)
    projs = workloads.config3(T)
    devs = [DeviceProj(p) for p in projs]
    lordba.adapter_forward_batched([d.proj() for d in devs], T, lordba.BF16)
    for p, d in zip(projs, devs):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16",
                     "config3/T=%d/%s/%s" % (T, p.name, vname))


@pytest.mark.parametrize("T,d_in,d_out,r,dtype", [
    (1, 11008, 4096, 16, "bf16"), (8, 11008, 4096, 16, "bf16"), (33, 11008, 4096, 16, "bf16"),
    (100, 11008, 4096, 16, "bf16"), (300, 11008, 4096, 16, "bf16"), (500, 11008, 4096, 16, "bf16"),
    (8, 8192, 1024, 64, "bf16"), (40, 8192 + 256, 512, 8, "bf16"), (8, 16384, 2048, 32, "f16"),
    (20, 11008, 4096, 12, "bf16"), (64, 11008, 4096, 16, "f16"),
])
def test_few_tokens_long_d_in_shared_first_product(oracle, T, d_in, d_out, r, dtype):
    """Few token tiles and a long d_in: the CTAs of a tile share the first product (Eq. 8, u = A_sign
    (s_in x)) as a cluster, each summing its part of d_in, parts added in a fixed order.  Every
    element against the oracle; twice the same bits; also with the x-ready promise."""
    p = workloads.make_projection(d_in, d_out, r, T, dtype, seed=9500 + T + r)
    a, b, c = DeviceProj(p), DeviceProj(p), DeviceProj(p)
    code = lordba.BF16 if dtype == "bf16" else lordba.F16
    assert lordba.query_variant([a.proj()], T, code) == [lordba.VARIANT_MMA]
    a.forward()
    b.forward()
    lordba.adapter_forward(c.x, c.packed_A, c.packed_B, c.s_in, c.s_r, c.s_out, c.y, r, x_ready=True)
    assert_close(torch_to_f64(a.y), oracle_forward(oracle, p), dtype, "shared first product T=%d r=%d" % (T, r))
    assert torch.equal(a.y, b.y) and torch.equal(a.y, c.y)
    assert lordba.device_status() == 0


def test_shared_first_product_gives_the_same_bits_every_time():
    """The partial sums cross the cluster in whatever order the CTAs finish and are added in rank
    order: 40 runs of a decode-sized layer call (different launch timing every time, the previous
    run's kernels still draining) give one result."""
    T = 8
    projs = workloads.config3(T)
    first = None
    for run in range(40):
        devs = [DeviceProj(p) for p in projs]
        lordba.adapter_forward_batched([d.proj() for d in devs], T, lordba.BF16)
        ys = [d.y for d in devs]
        if first is None:
            first = ys
        else:
            for a, b in zip(first, ys):
                assert torch.equal(a, b), "run %d differs" % run
    assert lordba.device_status() == 0


def test_few_tokens_segments_with_shared_first_product(oracle):
    """Per-projection token counts in a decode-sized batched call (one projection empty, one with
    fewer tiles than the others): the clusters of a projection's missing tiles leave together."""
    lengths = [40, 0, 7, 33]
    ps = [workloads.make_projection(11008, 4096, 16, 40, "bf16", seed=9600 + i) for i in range(4)]
    ds = [DeviceProj(p) for p in ps]
    y0 = [d.y.clone() for d in ds]
    lordba.adapter_forward_segments([d.proj() for d in ds], lengths, lordba.BF16)
    for p, d, n, y in zip(ps, ds, lengths, y0):
        rows = np.arange(n)
        if n:
            assert_close(torch_to_f64(d.y[:n]), oracle_forward(oracle, p, rows=rows), "bf16", "segment of %d" % n,
                         scale_from=oracle_forward(oracle, p))
        assert torch.equal(d.y[n:], y[n:])
    assert lordba.device_status() == 0


@pytest.mark.parametrize("r", [8, 16, 32, 64])
def test_config4_one_layer_with_outliers(oracle, r):
    """One layer of the 32-layer set at a reduced T that still spans several token tiles and a
    ragged tail, every element checked; the full 224-projection launch is checked on samples
    in test_config4_full_set_sampled."""
    T = 300
    projs = workloads.config4_layer(0, T, r)
    devs = [DeviceProj(p) for p in projs]
    lordba.adapter_forward_batched([d.proj() for d in devs], T, lordba.BF16)
    for p, d in zip(projs, devs):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "config4/r=%d/%s" % (r, p.name))


@functools.lru_cache(maxsize=1)
def _config4_activations(T):
    """Activations of the full-set test for one T: x drawn once per layer shape (with the 1 % outlier
    channels), y once per output width; shared by the rank sweep so that host generation stays short."""
    rng = np.random.default_rng(99)
    base = {}
    for name, d_in, d_out in workloads.LAYER_PROJECTIONS:
        if d_in not in base:
            base[d_in] = workloads.make_projection(d_in, 8, 8, T, "bf16", seed=4900 + d_in, outlier_frac=0.01)
    # the first and the last token tile in full, plus random rows: at least 64 rows per projection
    rows = np.unique(np.concatenate([np.arange(16), np.arange(T - 16, T), rng.integers(0, T, size=40)]))
    assert len(rows) >= 64
    x_bits = {d_in: b.x for d_in, b in base.items()}
    x_f64 = {d_in: b.x_f64()[rows] for d_in, b in base.items()}
    y0 = {d: workloads.to_bf16_bits(rng.standard_normal((T, d), dtype=np.float32))
          for d in (workloads.HIDDEN, workloads.FFN)}
    y0_f64 = {d: workloads.bf16_bits_to_f32(a[rows]).astype(np.float64) for d, a in y0.items()}
    return rows, x_bits, x_f64, y0, y0_f64


@pytest.mark.parametrize("T", [2048, 4096])
@pytest.mark.parametrize("r", [8, 16, 32, 64])
def test_config4_full_set_sampled(oracle, r, T):
    """All 224 projections in one batched call at full T, every point of the rank sweep, on the
    kernels the library takes by itself (the streaming kernel in launches of 24 projections for
    r <= 16, the tcgen05 kernel in launches of up to 96 for r = 32 and 64).  Activations are drawn
    once per layer shape (three x tensors, shared read-only by the projections that take them);
    every projection has its own carriers, scales and y.  The oracle checks at least 64 token rows
    of every projection (the first and the last tile in full plus random rows)."""
    dev = torch.device("cuda:0")
    rows, x_bits, x_f64, y0, y0_f64 = _config4_activations(T)
    x_dev = {d_in: np_to_torch(a, "bf16", dev) for d_in, a in x_bits.items()}
    y0_dev = {d: np_to_torch(a, "bf16", dev) for d, a in y0.items()}

    keep, descs, checks = [], [], []
    for layer in range(workloads.N_LAYERS):
        for pi, (name, d_in, d_out) in enumerate(workloads.LAYER_PROJECTIONS):
            small = workloads.make_projection(d_in, d_out, r, 1, "bf16", seed=5000 + 7 * layer + pi)
            A = torch.from_numpy(small.A_sign).to(dev)
            B = torch.from_numpy(small.B_sign).to(dev)
            t = dict(pa=lordba.pack_signs(A, 0), pb=lordba.pack_signs(B, 1),
                     s_in=torch.from_numpy(small.s_in).to(dev), s_r=torch.from_numpy(small.s_r).to(dev),
                     s_out=torch.from_numpy(small.s_out).to(dev), y=y0_dev[d_out].clone())
            keep.append(t)
            descs.append(lordba.make_proj(x_dev[d_in], t["pa"], t["pb"], t["s_in"], t["s_r"],
                                          t["s_out"], t["y"], r))
            checks.append((small, d_in, d_out, t))
    # the route the library takes by itself at this point of the sweep
    fams = set(lordba.query_variant(descs, T, lordba.BF16))
    assert fams == ({lordba.VARIANT_TC} if r >= 32 else {lordba.VARIANT_MMA}), fams
    n0 = lordba.launch_count()
    lordba.adapter_forward_batched(descs, T, lordba.BF16)
    torch.cuda.synchronize()
    assert lordba.launch_count() - n0 == (3 if r >= 32 else 10)
    rows_t = torch.from_numpy(rows).to(dev)
    for i, (small, d_in, d_out, t) in enumerate(checks):
        got = torch_to_f64(t["y"][rows_t])
        want = oracle.adapter_forward(x_f64[d_in], small.A_sign, small.B_sign,
                                      small.s_in.astype(np.float64), small.s_r.astype(np.float64),
                                      small.s_out.astype(np.float64), y0_f64[d_out])
        assert_close(got, want, "bf16", "config4 full r=%d T=%d proj %d" % (r, T, i))


# ---------------------------------------------------------------- shapes, pitches, edge cases

SHAPES = [
    # T, d_in, d_out, r
    (1, 8, 8, 1), (3, 33, 17, 3), (5, 100, 60, 5), (17, 256, 256, 8), (64, 512, 384, 16),
    (129, 1000, 1032, 16), (130, 4096, 1376, 32), (257, 2048, 520, 64), (9, 64, 64, 64),
    (40, 11008, 128, 16), (260, 640, 11008, 8), (1, 4096, 4096, 16), (200, 4104, 4104, 24),
    (33, 72, 200, 40), (128, 128, 128, 16), (127, 192, 136, 8), (385, 1024, 768, 48),
    # ranks below 8 on shapes that the streaming kernel takes (several B_sign rows per byte)
    (300, 1024, 768, 4), (70, 512, 1536, 2), (33, 1024, 512, 1), (1100, 4096, 4096, 4), (9, 11008, 4096, 4),
    # other ranks that are not multiples of 8 (B_sign rows start at any bit)
    (150, 1024, 1024, 12), (77, 512, 1024, 3), (260, 4096, 512, 20), (40, 1024, 1024, 57), (64, 512, 512, 63),
    (31, 2048, 1024, 6), (500, 4096, 4096, 28),
]


@pytest.mark.parametrize("T,d_in,d_out,r", SHAPES)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_shapes_every_element(oracle, T, d_in, d_out, r, dtype, vname, variant):
    lordba.set_variant(variant)
    p = workloads.make_projection(d_in, d_out, r, T, dtype, seed=T * 31 + d_in + r, scales="tiny")
    d = DeviceProj(p)
    d.forward()
    assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), dtype,
                 "shape %s %s %s" % ((T, d_in, d_out, r), dtype, vname))


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("ldx_pad,ldy_pad", [(8, 16), (3, 5), (64, 0), (0, 24)])
@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_row_pitch_and_guard_bands(oracle, dtype, ldx_pad, ldy_pad, vname, variant):
    """ldx > d_in, ldy > d_out: the padding columns of y must come back untouched."""
    lordba.set_variant(variant)
    T, d_in, d_out, r = 150, 520, 392, 16
    p = workloads.make_projection(d_in, d_out, r, T, dtype, seed=77, scales="tiny")
    d = DeviceProj(p, ldx=d_in + ldx_pad, ldy=d_out + ldy_pad)
    d.forward()
    assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), dtype, "pitch %s" % vname)
    if ldy_pad:
        pad = d.y_buf[:, d_out:]
        assert bool((pad == -3.0).all()), "padding columns of y were written"


@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_unaligned_views(oracle, vname, variant):
    """x and y that start 2 bytes (bf16) into an allocation: no 16-byte alignment anywhere."""
    lordba.set_variant(variant)
    T, d_in, d_out, r = 70, 264, 200, 16
    p = workloads.make_projection(d_in, d_out, r, T, "bf16", seed=78, scales="tiny")
    dev = torch.device("cuda:0")
    xb = torch.zeros(T * d_in + 8, dtype=torch.bfloat16, device=dev)
    yb = torch.zeros(T * d_out + 8, dtype=torch.bfloat16, device=dev)
    x = xb[1:1 + T * d_in].view(T, d_in)
    y = yb[1:1 + T * d_out].view(T, d_out)
    x.copy_(np_to_torch(p.x, "bf16", dev))
    y.copy_(np_to_torch(p.y, "bf16", dev))
    d = DeviceProj(p)
    lordba.adapter_forward(x, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, y, r)
    assert_close(torch_to_f64(y), oracle_forward(oracle, p), "bf16", "unaligned " + vname)
    assert float(yb[0]) == 0.0 and float(yb[-1]) == 0.0


def test_empty_batch_and_zero_tokens():
    p = workloads.make_projection(64, 64, 8, 4, "bf16", seed=1)
    d = DeviceProj(p)
    before = d.y.clone()
    n0 = lordba.launch_count()
    lordba.adapter_forward(d.x[:0], d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, d.y[:0], 8)
    lordba.adapter_forward_batched([], 4, lordba.BF16)
    torch.cuda.synchronize()
    assert lordba.launch_count() == n0
    assert torch.equal(d.y, before)


# ---------------------------------------------------------------- properties the method fixes

@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_canonical_adapter_is_integer_exact(oracle, dtype, vname, variant):
    """Unit input/output scales, a power-of-two rank scale and small-integer x: every partial
    sum is exactly representable, so the kernels must agree with the oracle bit for bit."""
    lordba.set_variant(variant)
    rng = np.random.default_rng(5)
    T, d_in, d_out, r = 140, 512, 264, 16
    p = workloads.make_projection(d_in, d_out, r, T, dtype, seed=5, scales="tiny")
    xi = rng.integers(-2, 3, size=(T, d_in)).astype(np.float32)
    yi = rng.integers(-8, 9, size=(T, d_out)).astype(np.float32)
    p.x = workloads.to_bf16_bits(xi) if dtype == "bf16" else xi.astype(np.float16) if dtype == "f16" else xi
    p.y = workloads.to_bf16_bits(yi) if dtype == "bf16" else yi.astype(np.float16) if dtype == "f16" else yi
    p.s_in = np.ones(d_in, np.float32)
    p.s_out = np.ones(d_out, np.float32)
    p.s_r = np.full(r, 2.0 ** -6, np.float32)
    want = oracle_forward(oracle, p)
    if dtype == "bf16":
        # keep only outputs that a bf16 can hold exactly (|v| * 64 an integer below 2^8)
        exact = np.abs(want * 64) <= 255
        assert exact.mean() > 0.2
    elif dtype == "f16":
        exact = np.abs(want * 64) <= 2047            # 11 significant bits
        assert exact.mean() > 0.9
    else:
        exact = np.ones_like(want, bool)
    d = DeviceProj(p)
    d.forward()
    got = torch_to_f64(d.y)
    assert np.array_equal(got[exact], want[exact])


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_zero_rank_scale_leaves_y_untouched_and_runs_are_deterministic(oracle, dtype, vname, variant):
    lordba.set_variant(variant)
    p = workloads.make_projection(1024, 776, 16, 333, dtype, seed=6)
    d = DeviceProj(p)
    y0 = d.y.clone()
    keep = d.s_r.clone()
    d.s_r.zero_()
    d.forward()
    assert torch.equal(d.y, y0)
    d.s_r.copy_(keep)
    d.forward()
    first = d.y.clone()
    d.reset_y()
    d.forward()
    assert torch.equal(d.y, first)


@pytest.mark.parametrize("vname,variant", VARIANTS)
@skip_unsupported
def test_padded_rank_matches(oracle, vname, variant):
    """An r=8 adapter padded to r=16 with zero rank scales gives the same output (bf16 path)."""
    lordba.set_variant(variant)
    rng = np.random.default_rng(8)
    p8 = workloads.make_projection(768, 520, 8, 200, "bf16", seed=8)
    p16 = workloads.make_projection(768, 520, 16, 200, "bf16", seed=8)
    p16.x, p16.y = p8.x, p8.y
    p16.A_sign[:8], p16.B_sign[:, :8] = p8.A_sign, p8.B_sign
    p16.s_in, p16.s_out = p8.s_in, p8.s_out
    p16.s_r = np.concatenate([p8.s_r, np.zeros(8, np.float32)])
    a, b = DeviceProj(p8), DeviceProj(p16)
    a.forward()
    b.forward()
    want = oracle_forward(oracle, p8)
    assert_close(torch_to_f64(a.y), want, "bf16", "r=8 " + vname)
    assert_close(torch_to_f64(b.y), want, "bf16", "r=16 padded " + vname)


def test_overlapping_run_of_calls_q_k_v(oracle):
    """Three adapters on the same x writing three y buffers, the second and third declared
    independent of the calls before them (LORDBA_PROJ_OVERLAP), then a plain call that reads one
    of those outputs as its x: every result must still match the oracle."""
    T = 2048
    base = workloads.make_projection(4096, 4096, 16, T, "bf16", seed=60)
    projs = [base] + [workloads.make_projection(4096, 4096, 16, T, "bf16", seed=61 + i) for i in range(2)]
    for p in projs[1:]:
        p.x = base.x
    devs = [DeviceProj(p) for p in projs]
    for i, d in enumerate(devs):
        lordba.adapter_forward(devs[0].x, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, d.y, 16,
                               overlap=(i > 0))
    # dependent follow-up: x = the first call's output, no flag
    nxt = workloads.make_projection(4096, 4096, 16, T, "bf16", seed=70)
    dn = DeviceProj(nxt)
    lordba.adapter_forward(devs[0].y, dn.packed_A, dn.packed_B, dn.s_in, dn.s_r, dn.s_out, dn.y, 16)
    torch.cuda.synchronize()
    for p, d in zip(projs, devs):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "overlap run " + str(p.meta["seed"]))
    nxt.x = devs[0].y.view(torch.int16).cpu().numpy().view(np.uint16)
    assert_close(torch_to_f64(dn.y), oracle_forward(oracle, nxt), "bf16", "call after the run")


def test_host_buffer_entry(oracle):
    p = workloads.make_projection(1024, 1536, 16, 300, "bf16", seed=9)
    d = DeviceProj(p)
    xh = np_to_torch(p.x, "bf16", "cpu").pin_memory()
    yh = np_to_torch(p.y, "bf16", "cpu").pin_memory()
    ws = torch.empty(lordba.host_workspace_bytes(p.T, p.d_in, p.d_out, lordba.BF16),
                     dtype=torch.uint8, device="cuda:0")
    lordba.adapter_forward_host(xh, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, yh, p.r, ws)
    torch.cuda.synchronize()
    assert_close(yh.to(torch.float64).numpy(), oracle_forward(oracle, p), "bf16", "host entry")


def test_carriers_packed_by_oracle_and_by_library_agree(oracle):
    p = workloads.make_projection(520, 392, 16, 40, "bf16", seed=10)
    a = DeviceProj(p, pack_on_gpu=True)
    b = DeviceProj(p, pack_on_gpu=False, oracle=oracle)
    assert torch.equal(a.packed_A, b.packed_A) and torch.equal(a.packed_B, b.packed_B)


# ---------------------------------------------------------------- multi-envelope adapters (Eq. 4, ell > 1)

def _ell_inputs(d_in, d_out, r, T, dtype, ell, seed):
    base = workloads.make_projection(d_in, d_out, r, T, dtype, seed=seed)
    rng = np.random.default_rng(seed + 77)
    s_in = np.exp(rng.normal(0.0, 0.5, size=(ell, d_in))).astype(np.float32)
    s_r = (64.0 * np.abs(rng.normal(0.0, 0.02, size=(ell, r)))).astype(np.float32)
    s_out = np.exp(rng.normal(0.0, 0.5, size=(ell, d_out))).astype(np.float32)
    return base, s_in, s_r, s_out


ELL_SHAPES = [
    # T, d_in, d_out, r, ell
    (70, 256, 192, 8, 2), (300, 1024, 768, 16, 2), (33, 200, 136, 24, 3), (150, 4096, 1024, 16, 4),
    (2048, 4096, 4096, 16, 2),
    # every envelope count the streaming kernel takes in one pass (ell * padded rank <= 64) ...
    (200, 1024, 768, 4, 2), (130, 512, 1024, 8, 8), (90, 1024, 512, 16, 3), (300, 768, 1024, 8, 5),
    (100, 1024, 768, 12, 3), (2048, 4096, 4096, 4, 2), (2048, 4096, 4096, 16, 4),
    # ... and in several passes over x (ell * padded rank > 64)
    (300, 1024, 1024, 32, 4), (64, 512, 512, 64, 2), (200, 1024, 1024, 32, 8), (100, 512, 512, 64, 8),
    (150, 1024, 512, 20, 5), (77, 512, 1024, 40, 3),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("T,d_in,d_out,r,ell", ELL_SHAPES)
def test_multi_envelope_forward(oracle, dtype, T, d_in, d_out, r, ell):
    if dtype != "bf16" and T > 1000:
        pytest.skip("full-size case is checked in bf16 only")
    base, s_in, s_r, s_out = _ell_inputs(d_in, d_out, r, T, dtype, ell, seed=90 + ell + r)
    d = DeviceProj(base)
    dev = d.x.device
    t_in, t_r, t_out = (torch.from_numpy(v).to(dev) for v in (s_in, s_r, s_out))
    if dtype != "f32" and d_in % 64 == 0 and d_out % 64 == 0:
        # every envelope count and rank runs on the tensor cores
        p = lordba.make_proj(d.x, d.packed_A, d.packed_B, t_in, t_r, t_out, d.y, r)
        assert lordba.query_variant([p], T, lordba.BF16 if dtype == "bf16" else lordba.F16) == [lordba.VARIANT_MMA]
    lordba.adapter_forward_ell(d.x, d.packed_A, d.packed_B, t_in, t_r, t_out, d.y, r)
    want = oracle.adapter_forward_ell(base.x_f64(), base.A_sign, base.B_sign, s_in.astype(np.float64),
                                      s_r.astype(np.float64), s_out.astype(np.float64), base.y_f64())
    assert_close(torch_to_f64(d.y), want, dtype, "ell=%d r=%d %s" % (ell, r, dtype))


TC_ELL_SHAPES = [
    # T, d_in, d_out, r  (two envelopes; ell * r <= 64).  Few tokens: the feature axes are split over a
    # cluster and the partial sums of both envelopes cross it; widths that are not multiples of 64
    # end in a ragged chunk; 2048 + 40 tokens: full tiles, one CTA per tile, and a short last tile
    (300, 1024, 768, 32), (70, 256, 192, 8), (200, 512, 512, 24), (130, 1000, 520, 16), (1, 512, 512, 32),
    (2048 + 40, 4096, 1024, 32), (1500, 1024, 4096, 16),
]


@pytest.mark.parametrize("dtype", ["bf16", "f16", "f16-exact"])
@pytest.mark.parametrize("T,d_in,d_out,r", TC_ELL_SHAPES)
def test_two_envelopes_on_the_tcgen05_kernel(oracle, dtype, T, d_in, d_out, r):
    """Two-envelope adapters (Def. 1 / Eq. 4) with the tcgen05 kernel pinned: every element against the
    oracle, in bfloat16, in float16, and in float16 with input scales that are float16 values."""
    io = "bf16" if dtype == "bf16" else "f16"
    if io != "bf16" and T > 1000:
        pytest.skip("full-size cases are checked in bf16 only")
    base, s_in, s_r, s_out = _ell_inputs(d_in, d_out, r, T, io, 2, seed=400 + r + d_in % 97)
    flags = 0
    if dtype == "f16-exact":
        s_in = s_in.astype(np.float16).astype(np.float32)
        flags = lordba.PROJ_SCALES_F16
    d = DeviceProj(base)
    t_in, t_r, t_out = (torch.from_numpy(v).to(d.x.device) for v in (s_in, s_r, s_out))
    p = lordba.make_proj(d.x, d.packed_A, d.packed_B, t_in, t_r, t_out, d.y, r, flags)
    code = lordba.BF16 if io == "bf16" else lordba.F16
    lordba.set_variant(lordba.VARIANT_TC)
    assert lordba.query_variant([p], T, code) == [lordba.VARIANT_TC]
    n0 = lordba.launch_count()
    lordba.adapter_forward_batched([p], T, code)
    assert lordba.launch_count() - n0 == 1
    want = oracle.adapter_forward_ell(base.x_f64(), base.A_sign, base.B_sign, s_in.astype(np.float64),
                                      s_r.astype(np.float64), s_out.astype(np.float64), base.y_f64())
    assert_close(torch_to_f64(d.y), want, io, "tcgen05 ell=2 r=%d %s" % (r, dtype))
    assert lordba.device_status() == 0


def test_two_envelope_segments_and_mixed_counts_on_the_tcgen05_kernel(oracle):
    """One pinned tcgen05 call with per-projection token counts whose projections have one and two
    envelopes at several ranks: one launch per (envelope count, rank), every element checked."""
    specs = [(1024, 512, 32, 2, 300), (1024, 512, 32, 1, 77), (512, 768, 16, 2, 0), (768, 1024, 16, 2, 150),
             (512, 512, 64, 1, 130), (1024, 1024, 8, 2, 200)]
    T = max(t for *_, t in specs)
    devs, wants, keep = [], [], []
    for i, (d_in, d_out, r, ell, rows) in enumerate(specs):
        base, s_in, s_r, s_out = _ell_inputs(d_in, d_out, r, T, "bf16", ell, seed=760 + i)
        d = DeviceProj(base)
        ts = [torch.from_numpy(v if ell > 1 else v[0]).to(d.x.device) for v in (s_in, s_r, s_out)]
        keep.append(ts)
        devs.append((d, lordba.make_proj(d.x, d.packed_A, d.packed_B, ts[0], ts[1], ts[2], d.y, r)))
        want = base.y_f64().copy()
        want[:rows] = oracle.adapter_forward_ell(base.x_f64()[:rows], base.A_sign, base.B_sign, s_in.astype(np.float64),
                                                 s_r.astype(np.float64), s_out.astype(np.float64), base.y_f64()[:rows])
        wants.append(want)
    lordba.set_variant(lordba.VARIANT_TC)
    n0 = lordba.launch_count()
    lordba.adapter_forward_segments([p for _, p in devs], [t for *_, t in specs], lordba.BF16)
    assert lordba.launch_count() - n0 == 5          # (2,32) (1,32) (2,16) (1,64) (2,8); the empty one launches nothing
    for (d, _), want, spec in zip(devs, wants, specs):
        assert_close(torch_to_f64(d.y), want, "bf16", "tcgen05 segments %s" % (spec,))


def test_multi_envelope_batched_with_mixed_envelope_counts(oracle):
    """One batched call whose projections differ in envelope count and rank: one launch per kind,
    every element against the oracle; and the zero-envelope embedding (an extra envelope with
    zero rank scales changes nothing, Eq. iota-embed)."""
    T = 150
    specs = [(1024, 512, 16, 1), (1024, 512, 16, 3), (512, 768, 8, 8), (768, 1024, 32, 2), (512, 512, 64, 3)]
    devs, wants, keep = [], [], []
    for i, (d_in, d_out, r, ell) in enumerate(specs):
        base, s_in, s_r, s_out = _ell_inputs(d_in, d_out, r, T, "bf16", ell, seed=700 + i)
        d = DeviceProj(base)
        ts = [torch.from_numpy(v if ell > 1 else v[0]).to(d.x.device) for v in (s_in, s_r, s_out)]
        keep.append(ts)
        devs.append((d, lordba.make_proj(d.x, d.packed_A, d.packed_B, ts[0], ts[1], ts[2], d.y, r)))
        wants.append(oracle.adapter_forward_ell(base.x_f64(), base.A_sign, base.B_sign, s_in.astype(np.float64),
                                                s_r.astype(np.float64), s_out.astype(np.float64), base.y_f64()))
    n0 = lordba.launch_count()
    lordba.adapter_forward_batched([p for _, p in devs], T, lordba.BF16)
    assert lordba.launch_count() - n0 == len(specs)
    for (d, _), want, spec in zip(devs, wants, specs):
        assert_close(torch_to_f64(d.y), want, "bf16", "mixed envelope counts %s" % (spec,))
    base, s_in, s_r, s_out = _ell_inputs(1024, 768, 16, 200, "bf16", 2, seed=720)
    a, b = DeviceProj(base), DeviceProj(base)
    t = lambda v: torch.from_numpy(np.ascontiguousarray(v)).to(a.x.device)
    pad = lambda v: np.concatenate([v, np.zeros_like(v[:1])]) if v.shape[1] == 16 else np.concatenate([v, np.ones_like(v[:1])])
    lordba.adapter_forward_ell(a.x, a.packed_A, a.packed_B, t(s_in), t(s_r), t(s_out), a.y, 16)
    lordba.adapter_forward_ell(b.x, b.packed_A, b.packed_B, t(pad(s_in)), t(pad(s_r)), t(pad(s_out)), b.y, 16)
    assert torch.equal(a.y, b.y)


def test_multi_envelope_with_one_envelope_equals_plain_call(oracle):
    base, s_in, s_r, s_out = _ell_inputs(1024, 1024, 16, 200, "bf16", 1, seed=95)
    a, b = DeviceProj(base), DeviceProj(base)
    dev = a.x.device
    t = lambda v: torch.from_numpy(v).to(dev)
    lordba.adapter_forward_ell(a.x, a.packed_A, a.packed_B, t(s_in), t(s_r), t(s_out), a.y, 16)
    lordba.adapter_forward(b.x, b.packed_A, b.packed_B, t(s_in[0]), t(s_r[0]), t(s_out[0]), b.y, 16)
    assert torch.equal(a.y, b.y)


# ---------------------------------------------------------------- the x-ready promise

@pytest.mark.parametrize("T,d_in,d_out,r", [(2048, 4096, 4096, 16), (300, 1024, 768, 32), (2048, 11008, 4096, 16), (40, 512, 512, 8)])
def test_x_ready_chain_on_one_y(oracle, T, d_in, d_out, r):
    """LORDBA_PROJ_X_READY (Eq. 2: the adapter call follows the work that produced y): three calls
    in a row update the SAME y from three inputs and adapters that were final beforehand, the second
    and third with the promise, so each starts on its x while its predecessor still writes y and
    must not touch y before that one is complete.  The result equals, bit for bit and on every one
    of 10 rounds, that of the same chain without the promise (a call that read y early would lose an
    update), which is checked against the oracle chain element by element."""
    ps = [workloads.make_projection(d_in, d_out, r, T, "bf16", seed=9300 + i) for i in range(3)]
    ds = [DeviceProj(p) for p in ps]
    y0 = ds[0].y.clone()
    want = ps[0].y_f64()
    bound = np.zeros_like(want)
    for p in ps:
        # each call rounds y to bfloat16 once and the oracle chain does the same between the calls.
        # Where the two sides round an intermediate y to different neighbours they leave that call
        # a whole bfloat16 step apart (2^-7 |y|, twice the bound of a single call), and every
        # call adds its own share, relative to what y holds after it
        want = oracle.adapter_forward(p.x_f64(), p.A_sign, p.B_sign, p.s_in.astype(np.float64), p.s_r.astype(np.float64),
                                      p.s_out.astype(np.float64), want)
        bound += 2.0 ** -7 * np.abs(want) + 2.0 ** -12 * np.sqrt(np.mean(want ** 2))
        want = torch.from_numpy(want).to(torch.bfloat16).to(torch.float64).numpy()

    def chain(promise):
        y = y0.clone()
        torch.cuda.current_stream().synchronize()
        for i, d in enumerate(ds):
            lordba.adapter_forward(d.x, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, y, r, x_ready=promise and i > 0)
        return y

    plain = chain(False)
    for rnd in range(10):
        assert torch.equal(chain(True), plain), "round %d differs from the chain without the promise" % rnd
    err = np.abs(torch_to_f64(plain) - want)
    assert np.all(err <= bound), float((err / bound).max())
    assert lordba.device_status() == 0


def test_x_ready_after_other_work_and_with_the_other_flags(oracle):
    """The promise after a kernel that is not the library's (y filled by a copy just before the
    call), on a batched call, and next to LORDBA_PROJ_OVERLAP (then ignored): every element."""
    T = 300
    ps = [workloads.make_projection(1024, 768, 16, T, "bf16", seed=9400 + i) for i in range(3)]
    ds = [DeviceProj(p) for p in ps]
    for d in ds:
        d.y.copy_(d.y.clone())                     # y "produced" on the stream right before the call
    flags = [lordba.PROJ_X_READY, lordba.PROJ_X_READY, lordba.PROJ_X_READY | lordba.PROJ_OVERLAP]
    projs = [lordba.make_proj(d.x, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, d.y, 16, f) for d, f in zip(ds, flags)]
    lordba.adapter_forward_batched(projs[:2], T, lordba.BF16)
    lordba.adapter_forward_batched(projs[2:], T, lordba.BF16)
    for p, d in zip(ps, ds):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "x-ready " + str(p.meta["seed"]))


# ---------------------------------------------------------------- multi-adapter batches (segments)

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d_in,d_out,r,lengths", [(1024, 768, 16, (100, 17, 0, 583)), (4096, 4096, 16, (256,) * 8),
                                                    (520, 392, 8, (1, 2, 3)), (2048, 1024, 32, (130, 130))])
def test_segments_each_with_its_own_adapter(oracle, dtype, d_in, d_out, r, lengths):
    """One x / y matrix, consecutive row segments, a different adapter per segment (the last
    segment reuses the first adapter): every segment must match the oracle run on its rows."""
    if dtype == "f32" and d_in == 4096:
        pytest.skip("full-size case is checked in bf16 only")
    T = sum(lengths)
    base = workloads.make_projection(d_in, d_out, r, T, dtype, seed=300 + r)
    n_adapters = max(1, len(lengths) - 1)
    adapters = [workloads.make_projection(d_in, d_out, r, 1, dtype, seed=310 + i) for i in range(n_adapters)]
    dev = torch.device("cuda:0")
    x = np_to_torch(base.x, dtype, dev)
    y = np_to_torch(base.y, dtype, dev)
    dads = [DeviceProj(a) for a in adapters]
    segs, want = [], base.y_f64().copy()
    start = 0
    for i, n in enumerate(lengths):
        a, da = adapters[i % n_adapters], dads[i % n_adapters]
        lo = min(start, T - 1)                      # an empty segment still needs a well-formed pointer
        segs.append(lordba.make_proj(x[lo:lo + max(n, 1)], da.packed_A, da.packed_B, da.s_in, da.s_r, da.s_out,
                                     y[lo:lo + max(n, 1)], r))
        if n:
            rows = slice(start, start + n)
            want[rows] = oracle.adapter_forward(base.x_f64()[rows], a.A_sign, a.B_sign, a.s_in.astype(np.float64),
                                                a.s_r.astype(np.float64), a.s_out.astype(np.float64),
                                                base.y_f64()[rows])
        start += n
    lordba.adapter_forward_segments(segs, lengths, lordba.BF16 if dtype == "bf16" else lordba.F32)
    assert_close(torch_to_f64(y), want, dtype, "segments %s %s" % (lengths, dtype))


# ---------------------------------------------------------------- the adjoint is the same path with the roles swapped

def test_adjoint_is_a_forward_with_swapped_carriers(oracle):
    """dX = ((dY D_gamma) B2^T D_beta) B1^T D_alpha (the backward of Eq. 8 with respect to X) is the
    forward of the adapter (A' = B_sign^T, B' = A_sign^T, s_in' = s_out, s_out' = s_in).  Checked
    two ways: against the oracle run on the swapped adapter, and through <dy, f(x)> = <f*(dy), x>."""
    T, d_in, d_out, r = 200, 1024, 768, 16
    p = workloads.make_projection(d_in, d_out, r, T, "bf16", seed=400)
    dy = workloads.to_bf16_bits(np.random.default_rng(401).standard_normal((T, d_out), dtype=np.float32))
    dev = torch.device("cuda:0")
    A_t = np.ascontiguousarray(p.B_sign.T)          # r x d_out: plays A_sign
    B_t = np.ascontiguousarray(p.A_sign.T)          # d_in x r: plays B_sign
    pa = lordba.pack_signs(torch.from_numpy(A_t).to(dev), 0)
    pb = lordba.pack_signs(torch.from_numpy(B_t).to(dev), 1)
    dy_dev = np_to_torch(dy, "bf16", dev)
    dx = torch.zeros(T, d_in, dtype=torch.bfloat16, device=dev)
    t = lambda v: torch.from_numpy(v).to(dev)
    lordba.adapter_forward(dy_dev, pa, pb, t(p.s_out), t(p.s_r), t(p.s_in), dx, r)
    dy64 = workloads.bf16_bits_to_f32(dy).astype(np.float64)
    want = oracle.adapter_forward(dy64, A_t, B_t, p.s_out.astype(np.float64), p.s_r.astype(np.float64),
                                  p.s_in.astype(np.float64), np.zeros((T, d_in)))
    assert_close(torch_to_f64(dx), want, "bf16", "adjoint")
    # inner-product identity with the oracle's forward of the original adapter (float64 on both sides)
    fx = oracle.adapter_forward(p.x_f64(), p.A_sign, p.B_sign, p.s_in.astype(np.float64), p.s_r.astype(np.float64),
                                p.s_out.astype(np.float64), np.zeros((T, d_out)))
    lhs, rhs = float((dy64 * fx).sum()), float((want * p.x_f64()).sum())
    assert abs(lhs - rhs) <= 1e-9 * max(abs(lhs), abs(rhs))


# ---------------------------------------------------------------- the export precision: float16

def test_scales_from_f16_is_exact():
    """Every half widens to the same float: subnormals, zeros, infinities and the largest finite value included."""
    rng = np.random.default_rng(5)
    bits = rng.integers(0, 1 << 16, size=5000, dtype=np.uint16)
    bits[:8] = [0x0000, 0x8000, 0x0001, 0x03ff, 0x0400, 0x7bff, 0x7c00, 0xfc00]
    h = bits.view(np.float16)
    keep = ~np.isnan(h)                          # NaN payloads are not compared
    dev = torch.from_numpy(bits.view(np.int16).copy()).view(torch.float16).cuda()
    got = lordba.scales_from_f16(dev).cpu().numpy()
    want = h.astype(np.float32)
    assert got.dtype == np.float32
    assert np.array_equal(got[keep].view(np.uint32), want[keep].view(np.uint32))
    assert np.isnan(got[~keep]).all()
    assert lordba.scales_from_f16(dev[:0]).numel() == 0


@pytest.mark.parametrize("r", [8, 16, 32, 64])
@pytest.mark.parametrize("scales_f16", [False, True])
def test_f16_activations_attention_full_size(oracle, r, scales_f16):
    """The attention projection at T = 2048 with float16 x and y: float32 scales (s_in as a pair of
    halves) and an adapter exported with float16 scales (one pass, flagged), every element."""
    p = workloads.make_projection(4096, 4096, r, 2048, "f16", seed=1000 + r, scales_f16=scales_f16)
    d = DeviceProj(p)
    assert d.flags() == (lordba.PROJ_SCALES_F16 if scales_f16 else 0)
    d.forward()
    assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "f16", "f16 attn r=%d exported=%s" % (r, scales_f16))


def test_f16_exported_adapter_loaded_from_half_storage(oracle):
    """An adapter stored with half-precision scales: widened by the library, used flagged and
    unflagged; both agree with the oracle run on the same half values."""
    p = workloads.make_projection(1024, 1536, 16, 333, "f16", seed=77, scales_f16=True)
    d = DeviceProj(p)
    for name in ("s_in", "s_r", "s_out"):
        stored = torch.from_numpy(getattr(p, name).astype(np.float16).view(np.int16).copy()).view(torch.float16).cuda()
        widened = lordba.scales_from_f16(stored)
        assert torch.equal(widened, getattr(d, name))
        setattr(d, name, widened)
    want = oracle_forward(oracle, p)
    for flagged in (True, False):
        d.reset_y()
        lordba.adapter_forward(d.x, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, d.y, p.r, scales_f16=flagged)
        assert_close(torch_to_f64(d.y), want, "f16", "exported adapter, flagged=%s" % flagged)


@pytest.mark.parametrize("c", [2.0 ** -8, 2.0 ** 6])
def test_f16_scale_gauge(oracle, c):
    """(c s_in, s_r / c, s_out) is the same adapter (c a power of two): small and large s_in
    stay within the float16 bound although s_in enters the tensor cores as halves."""
    p = workloads.make_projection(2048, 1024, 16, 200, "f16", seed=91)
    want = oracle_forward(oracle, p)
    p.s_in = (p.s_in * np.float32(c)).astype(np.float32)
    p.s_r = (p.s_r / np.float32(c)).astype(np.float32)
    d = DeviceProj(p)
    d.forward()
    assert_close(torch_to_f64(d.y), want, "f16", "gauge c=%g" % c)


def test_f16_mixed_batch_and_segments(oracle):
    """One batched call with flagged and unflagged projections of different rank, and a segmented call."""
    ps = [workloads.make_projection(di, do, r, 150, "f16", seed=300 + i, scales_f16=ex)
          for i, (di, do, r, ex) in enumerate([(512, 768, 16, True), (512, 768, 16, False), (1024, 256, 64, True),
                                               (200, 136, 24, False)])]
    ds = [DeviceProj(p) for p in ps]
    lordba.adapter_forward_batched([d.proj() for d in ds], 150, lordba.F16)
    for p, d in zip(ps, ds):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "f16", "f16 batched " + p.name)
    for d in ds:
        d.reset_y()
    tokens = [150, 0, 77, 150]
    lordba.adapter_forward_segments([d.proj() for d in ds], tokens, lordba.F16)
    for p, d, n in zip(ps, ds, tokens):
        got = torch_to_f64(d.y)
        want = oracle_forward(oracle, p)
        assert_close(got[:n], want[:n], "f16", "f16 segment " + p.name, scale_from=want)
        assert np.array_equal(got[n:], p.y_f64()[n:])


@pytest.mark.parametrize("r,scales_f16", [(64, False), (64, True), (24, True), (40, False)])
def test_f16_layer_on_the_tcgen05_kernel(oracle, r, scales_f16):
    """One decoder layer's seven projections with float16 activations, as the library runs them
    by itself and with the tcgen05 kernel pinned (full 128-token tiles plus a ragged last one):
    both forms of s_in (a pair of halves; one half, declared), ranks that are and are not
    multiples of 16.  Sampled rows: first tile, last (ragged) tile, random rows."""
    T = 2048 + 40
    rng = np.random.default_rng(11 + r)
    rows = np.unique(np.concatenate([np.arange(16), np.arange(T - 48, T), rng.integers(0, T, size=24)]))
    projs = [workloads.make_projection(di, do, r, T, "f16", seed=5000 + 7 * r + i, name=n, scales_f16=scales_f16,
                                       outlier_frac=0.01)
             for i, (n, di, do) in enumerate(workloads.LAYER_PROJECTIONS)]
    devs = [DeviceProj(p) for p in projs]
    lordba.adapter_forward_batched([d.proj() for d in devs], T, lordba.F16)
    rows_t = torch.from_numpy(rows).cuda()
    for p, d in zip(projs, devs):
        assert_close(torch_to_f64(d.y[rows_t]), oracle_forward(oracle, p, rows=rows), "f16",
                     "f16 layer r=%d %s" % (r, p.name))
    # and with the tcgen05 kernel pinned (the library's own choice only for ranks above 32 here)
    for d in devs:
        d.reset_y()
    lordba.set_variant(lordba.VARIANT_TC)
    lordba.adapter_forward_batched([d.proj() for d in devs], T, lordba.F16)
    for p, d in zip(projs, devs):
        assert_close(torch_to_f64(d.y[rows_t]), oracle_forward(oracle, p, rows=rows), "f16",
                     "f16 layer, tcgen05 pinned, r=%d %s" % (r, p.name))


def test_f16_mixed_scale_kinds_on_the_tcgen05_kernel(oracle):
    """One batched call, tcgen05 kernel pinned: projections with declared float16 scales and with
    float32 scales go out as separate launches that may overlap; every element checked."""
    T = 300
    ps = [workloads.make_projection(di, do, 64, T, "f16", seed=7000 + i, scales_f16=ex)
          for i, (di, do, ex) in enumerate([(1024, 768, True), (512, 1024, False), (768, 512, True), (1024, 1024, False)])]
    ds = [DeviceProj(p) for p in ps]
    lordba.set_variant(lordba.VARIANT_TC)
    lordba.adapter_forward_batched([d.proj() for d in ds], T, lordba.F16)
    for p, d in zip(ps, ds):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "f16", "f16 mixed tcgen05 " + str(p.meta["seed"]))


# ---------------------------------------------------------------- prepared calls and the kernel query

@pytest.mark.parametrize("kind", ["layer_r16", "layer_r64", "segments_r16", "mixed_families", "decode_r16"])
def test_planned_call_equals_plain_call(oracle, kind):
    """lordba_plan_init + lordba_adapter_forward_planned launch what the plain call launches: the
    same number of kernels, bit-identical y, and y matches the oracle; a plan can be replayed."""
    T = 300
    if kind == "layer_r16":
        projs = workloads.config4_layer(1, T, 16)
        tokens = T
    elif kind == "layer_r64":
        T = 2048 + 40                                     # enough 128-token tiles for the tcgen05 kernel
        projs = [workloads.make_projection(di, do, 64, T, "bf16", seed=8100 + i, name=n)
                 for i, (n, di, do) in enumerate(workloads.LAYER_PROJECTIONS[:4])]
        tokens = T
    elif kind == "segments_r16":
        projs = [workloads.make_projection(1024, 768, 16, T, "bf16", seed=8200 + i) for i in range(3)]
        tokens = [T, 0, 77]
    elif kind == "decode_r16":
        T = 8                                             # few tiles: launched as clusters that share the first product
        projs = workloads.config3(T)
        tokens = T
    else:
        # three kernel families in one call: widths that are not multiples of 64 (the tcgen05 kernel
        # takes them from 128 tokens up), a row pitch of 1001 elements (only the CUDA-core kernel),
        # and a shape for the streaming kernel
        projs = [workloads.make_projection(1000, 520, 16, T, "bf16", seed=8300),
                 workloads.make_projection(1001, 520, 16, T, "bf16", seed=8302),
                 workloads.make_projection(1024, 512, 16, T, "bf16", seed=8301)]
        tokens = T
    a = [DeviceProj(p) for p in projs]
    b = [DeviceProj(p) for p in projs]
    fams = lordba.query_variant([d.proj() for d in a], tokens, lordba.BF16)
    if kind == "layer_r64":
        assert set(fams) == {lordba.VARIANT_TC}
    if kind == "mixed_families":
        assert fams == [lordba.VARIANT_TC, lordba.VARIANT_FMA, lordba.VARIANT_MMA]
    if kind == "segments_r16":
        assert fams == [lordba.VARIANT_MMA, 0, lordba.VARIANT_MMA]
    plan = lordba.plan_init([d.proj() for d in b], tokens, lordba.BF16)
    n0 = lordba.launch_count()
    if isinstance(tokens, int):
        lordba.adapter_forward_batched([d.proj() for d in a], tokens, lordba.BF16)
    else:
        lordba.adapter_forward_segments([d.proj() for d in a], tokens, lordba.BF16)
    n1 = lordba.launch_count()
    lordba.adapter_forward_planned(plan)
    n2 = lordba.launch_count()
    torch.cuda.synchronize()
    assert n1 - n0 == n2 - n1 == plan.launches() and n1 > n0
    rows = [tokens] * len(projs) if isinstance(tokens, int) else tokens
    for p, da, db, n in zip(projs, a, b, rows):
        assert torch.equal(da.y, db.y)
        want = oracle_forward(oracle, p)
        assert_close(torch_to_f64(db.y)[:n], want[:n], "bf16", "planned " + kind, scale_from=want)
        assert np.array_equal(torch_to_f64(db.y)[n:], p.y_f64()[n:])
    # a second replay adds the adapter term once more
    for d in b:
        d.reset_y()
    lordba.adapter_forward_planned(plan)
    torch.cuda.synchronize()
    for da, db in zip(a, b):
        assert torch.equal(da.y, db.y)


def test_query_variant_shows_the_fallbacks():
    """The kernel family per projection, as the call would choose it: float32 activations, widths
    that are not multiples of 64, odd row pitches and unaligned scales go to the CUDA-core kernel."""
    T = 64
    ok = DeviceProj(workloads.make_projection(1024, 512, 16, T, "bf16", seed=1))
    f32 = DeviceProj(workloads.make_projection(1024, 512, 16, T, "f32", seed=2))
    odd = DeviceProj(workloads.make_projection(1000, 512, 16, T, "bf16", seed=3))
    pitch = DeviceProj(workloads.make_projection(1024, 512, 16, T, "bf16", seed=4), ldx=1024 + 3)
    assert lordba.query_variant([ok.proj()], T, lordba.BF16) == [lordba.VARIANT_MMA]
    assert lordba.query_variant([f32.proj()], T, lordba.F32) == [lordba.VARIANT_FMA]
    assert lordba.query_variant([odd.proj(), pitch.proj()], T, lordba.BF16) == [lordba.VARIANT_FMA] * 2
    # from one 128-token tile up the tcgen05 kernel takes the odd width; the odd pitch stays where it is
    odd2 = DeviceProj(workloads.make_projection(1000, 512, 16, 256, "bf16", seed=3))
    pitch2 = DeviceProj(workloads.make_projection(1024, 512, 16, 256, "bf16", seed=4), ldx=1024 + 3)
    assert lordba.query_variant([odd2.proj(), pitch2.proj()], 256, lordba.BF16) == [lordba.VARIANT_TC, lordba.VARIANT_FMA]
    big = [DeviceProj(workloads.make_projection(1024, 512, 64, 1, "bf16", seed=5))]
    x = torch.zeros(4096, 1024, dtype=torch.bfloat16, device="cuda:0")
    y = torch.zeros(4096, 512, dtype=torch.bfloat16, device="cuda:0")
    d = big[0]
    p = lordba.make_proj(x, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, y, 64)
    assert lordba.query_variant([p], 4096, lordba.BF16) == [lordba.VARIANT_TC]      # 32 tiles of 128 tokens
    assert lordba.query_variant([p], [2048], lordba.BF16) == [lordba.VARIANT_MMA]
    # two envelopes at rank 32 count as rank 64: the same rule
    two = lambda v: torch.stack([v, v]).contiguous()
    d32 = DeviceProj(workloads.make_projection(1024, 512, 32, 1, "bf16", seed=6))
    p2 = lordba.make_proj(x, d32.packed_A, d32.packed_B, two(d32.s_in), two(d32.s_r), two(d32.s_out), y, 32)
    assert lordba.query_variant([p2], 4096, lordba.BF16) == [lordba.VARIANT_TC]
    assert lordba.query_variant([p2], [2048], lordba.BF16) == [lordba.VARIANT_MMA]
    lordba.set_variant(lordba.VARIANT_TC)
    with pytest.raises(lordba.LordbaError) as e:
        lordba.query_variant([f32.proj()], T, lordba.F32)      # a pinned family that cannot take the call
    assert e.value.status == 2


def test_tcgen05_last_wave_dealt_from_the_other_end(oracle):
    """A launch of between three and five waves of tiles deals its last wave to the persistent CTAs
    in reverse order: 148 * 3 + 40 tiles of 128 tokens and a short one, two projections of
    different cost, every element against the oracle (a tile done twice or not at all would show)."""
    T = 128 * (74 * 3 + 20) + 5
    projs = [workloads.make_projection(512, 256, 64, T, "bf16", seed=9100),
             workloads.make_projection(256, 256, 64, T, "bf16", seed=9101)]
    devs = [DeviceProj(p) for p in projs]
    lordba.set_variant(lordba.VARIANT_TC)
    n0 = lordba.launch_count()
    lordba.adapter_forward_batched([d.proj() for d in devs], T, lordba.BF16)
    assert lordba.launch_count() - n0 == 1
    for p, d in zip(projs, devs):
        assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "tcgen05 four waves " + str(p.meta["seed"]))
    assert lordba.device_status() == 0


@pytest.mark.parametrize("r", [32, 64])
@pytest.mark.parametrize("pin", [False, True])
def test_segments_on_the_tcgen05_kernel(oracle, r, pin):
    """A multi-adapter batch at high rank: segments of different lengths (one empty, one shorter
    than a tile, one ending in a ragged tile), each with its own adapter, through the tcgen05
    kernel, which takes a token count per projection; every element against the oracle."""
    lengths = (1280, 0, 700, 50, 2100)
    d_in, d_out = 1024, 1536
    T = sum(lengths)
    base = workloads.make_projection(d_in, d_out, r, T, "bf16", seed=600 + r)
    adapters = [workloads.make_projection(d_in, d_out, r, 1, "bf16", seed=610 + i) for i in range(4)]
    dev = torch.device("cuda:0")
    x = np_to_torch(base.x, "bf16", dev)
    y = np_to_torch(base.y, "bf16", dev)
    dads = [DeviceProj(a) for a in adapters]
    segs, want, start = [], base.y_f64().copy(), 0
    for i, n in enumerate(lengths):
        a, da = adapters[i % 4], dads[i % 4]
        lo = min(start, T - 1)
        segs.append(lordba.make_proj(x[lo:lo + max(n, 1)], da.packed_A, da.packed_B, da.s_in, da.s_r, da.s_out,
                                     y[lo:lo + max(n, 1)], r))
        if n:
            rows = slice(start, start + n)
            want[rows] = oracle.adapter_forward(base.x_f64()[rows], a.A_sign, a.B_sign, a.s_in.astype(np.float64),
                                                a.s_r.astype(np.float64), a.s_out.astype(np.float64),
                                                base.y_f64()[rows])
        start += n
    if pin:
        lordba.set_variant(lordba.VARIANT_TC)
    fams = lordba.query_variant(segs, lengths, lordba.BF16)
    if pin or r > 32:
        assert set(fams) == {0, lordba.VARIANT_TC}
    lordba.adapter_forward_segments(segs, lengths, lordba.BF16)
    assert_close(torch_to_f64(y), want, "bf16", "tcgen05 segments r=%d" % r)
