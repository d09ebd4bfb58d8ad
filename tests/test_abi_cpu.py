"""The C-ABI library loads without a GPU, exports what the header declares, and
rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_24058_b200 import build, lordba
    build.build_library()
    return lordba.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "lordba.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lordba_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2605_24058_b200 import lordba
    declared = _declared_functions()
    assert len(declared) >= 16
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(lordba.exported_symbols()) == declared


def test_host_only_helpers(lib):
    from paper_2605_24058_b200 import lordba
    assert lordba.packed_words(16, 4096, 0) == 16 * 128
    assert lordba.packed_words(4096, 16, 1) == 2048
    assert lordba.packed_words(3, 33, 0) == 6 and lordba.packed_words(3, 65, 0) == 12
    assert lordba.packed_words(33, 3, 1) == 4
    assert lordba.packed_words(-1, 3, 0) == -1 and lordba.packed_words(1, 3, 2) == -1
    assert lordba.adapter_bits(3, 5, 2, 1) == 2 * 8 + 16 * 10          # Eq. 5 by hand
    assert lordba.adapter_bits(4096, 4096, 16, 1) == 16 * 8192 + 16 * (8192 + 16)
    assert lordba.status_string(0) == "ok" and "align" in lordba.status_string(3)
    assert "sm_100a" in lordba.version()
    assert lordba.host_workspace_bytes(2048, 4096, 4096, lordba.BF16) == 2 * 2048 * 4096 * 2


def test_library_helpers_match_oracle(lib, oracle):
    from paper_2605_24058_b200 import lordba
    for rows, cols in [(16, 4096), (8, 250), (1, 1), (64, 11008), (0, 5)]:
        for role in (0, 1):
            assert lordba.packed_words(rows, cols, role) == oracle.packed_words(rows, cols, role)
    for d_in, d_out, r, ell in [(4096, 11008, 16, 1), (256, 256, 8, 2), (11008, 4096, 64, 3)]:
        assert lordba.adapter_bits(d_in, d_out, r, ell) == oracle.adapter_bits(d_in, d_out, r, ell)


def _proj(lordba, **kw):
    base = dict(x=0x1000, packed_A=0x2000, packed_B=0x3000, s_in=0x4000, s_r=0x5000, s_out=0x6000,
                y=0x100000, d_in=64, d_out=64, ldx=64, ldy=64, r=8, flags=0)
    base.update(kw)
    return lordba.Proj(**base)


def test_bad_arguments_return_codes_without_launching(lib):
    """None of these reaches a launch, so they are safe without a device; the pointers
    are fake but well-formed."""
    from paper_2605_24058_b200 import lordba
    EINVAL, EUNSUP, EALIGN = 1, 2, 3
    call = lambda p, T=4, dt=lordba.BF16: lib.lordba_adapter_forward_ex(ctypes.byref(p), T, dt, None)
    before = lordba.launch_count()
    assert call(_proj(lordba, x=0)) == EINVAL
    assert call(_proj(lordba, y=0)) == EINVAL
    assert call(_proj(lordba, s_r=0)) == EINVAL
    assert call(_proj(lordba), T=-1) == EINVAL
    assert call(_proj(lordba, d_in=0)) == EINVAL
    assert call(_proj(lordba, ldx=63)) == EINVAL
    assert call(_proj(lordba, ldy=10)) == EINVAL
    assert call(_proj(lordba, flags=8)) == EINVAL
    assert call(_proj(lordba, flags=0x1000)) == EINVAL
    assert call(_proj(lordba, r=0)) == EUNSUP
    assert call(_proj(lordba, r=65)) == EUNSUP
    assert call(_proj(lordba), dt=9) == EUNSUP
    assert call(_proj(lordba, x=0x1001)) == EALIGN
    assert call(_proj(lordba, x=0x1002), dt=lordba.F32) == EALIGN
    assert call(_proj(lordba, packed_B=0x3002)) == EALIGN
    assert call(_proj(lordba, s_out=0x6001)) == EALIGN
    assert call(_proj(lordba, y=0x1010)) == EINVAL                     # y overlaps x
    assert lib.lordba_adapter_forward_ex(None, 4, lordba.BF16, None) == EINVAL
    # T = 0 is a no-op that succeeds
    assert call(_proj(lordba), T=0) == 0
    assert call(_proj(lordba, x=0, y=0), T=0) == 0
    assert call(_proj(lordba, r=0), T=0) == EUNSUP
    # batched: overlapping outputs, negative count
    two = (lordba.Proj * 2)(_proj(lordba), _proj(lordba, x=0x8000))
    assert lib.lordba_adapter_forward_batched(two, 2, 4, lordba.BF16, None) == EINVAL
    assert lib.lordba_adapter_forward_batched(two, -1, 4, lordba.BF16, None) == EINVAL
    # batched: one projection's x lies inside another projection's y
    chained = (lordba.Proj * 2)(_proj(lordba), _proj(lordba, x=0x100000, y=0x200000))
    assert lib.lordba_adapter_forward_batched(chained, 2, 4, lordba.BF16, None) == EINVAL
    assert lib.lordba_adapter_forward_batched(None, 0, 4, lordba.BF16, None) == 0
    # pack / unpack
    assert lib.lordba_pack_signs(0x1000, 4, 4, 5, 0x2000, None) == EUNSUP
    assert lib.lordba_pack_signs(None, 4, 4, 0, 0x2000, None) == EINVAL
    assert lib.lordba_pack_signs(0x1000, -4, 4, 0, 0x2000, None) == EINVAL
    assert lib.lordba_pack_signs(0x1000, 4, 4, 0, 0x2001, None) == EALIGN
    assert lib.lordba_pack_signs(0x1000, 0, 4, 0, 0x2000, None) == 0
    assert lib.lordba_unpack_signs(0x2000, 4, 4, 1, None, None) == EINVAL
    # host-buffer entry
    ws = lordba.host_workspace_bytes(4, 64, 64, lordba.BF16)
    args = (0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x9000, 4, 64, 64, 8, lordba.BF16)
    assert lib.lordba_adapter_forward_host(*args, 0x100000, ws - 1, None) == EINVAL
    assert lib.lordba_adapter_forward_host(*args, 0x100010, ws, None) == EALIGN
    assert lib.lordba_adapter_forward_host(*args, None, ws, None) == EINVAL
    # variant switch
    assert lib.lordba_set_variant(7) == EUNSUP
    assert lib.lordba_set_variant(lordba.VARIANT_FMA) == 0 and lordba.get_variant() == lordba.VARIANT_FMA
    assert lib.lordba_set_variant(lordba.VARIANT_AUTO) == 0
    assert lordba.launch_count() == before


def test_float16_arguments_and_inputs_without_launching(lib):
    """The float16 element type, the declared-scales flag and the scale widening entry: argument
    checks that return before any launch, and the seeded float16 inputs."""
    import numpy as np
    from paper_2605_24058_b200 import lordba, workloads
    EINVAL, EUNSUP, EALIGN = 1, 2, 3
    call = lambda p, T=4, dt=lordba.F16: lib.lordba_adapter_forward_ex(ctypes.byref(p), T, dt, None)
    assert call(_proj(lordba, flags=lordba.PROJ_SCALES_F16), T=0) == 0
    assert call(_proj(lordba, flags=lordba.PROJ_SCALES_F16 | lordba.PROJ_OVERLAP), T=0) == 0
    assert call(_proj(lordba, x=0x1001)) == EALIGN                    # 2-byte elements
    assert call(_proj(lordba, flags=lordba.PROJ_X_READY), T=0) == 0
    assert call(_proj(lordba, flags=8), T=0) == EINVAL
    assert lib.lordba_scales_from_f16(0x1000, 0x2000, -1, None) == EINVAL
    assert lib.lordba_scales_from_f16(None, 0x2000, 4, None) == EINVAL
    assert lib.lordba_scales_from_f16(0x1001, 0x2000, 4, None) == EALIGN
    assert lib.lordba_scales_from_f16(0x1000, 0x2002, 4, None) == EALIGN
    assert lib.lordba_scales_from_f16(None, None, 0, None) == 0
    # inputs: float16 x / y are the float32 draws rounded to nearest even; exported scales are
    # float16 values held in float32
    a = workloads.make_projection(64, 128, 8, 5, "f32", seed=3)
    b = workloads.make_projection(64, 128, 8, 5, "f16", seed=3, scales_f16=True)
    assert b.x.dtype == np.float16 and b.y.dtype == np.float16
    assert np.array_equal(b.x, a.x.astype(np.float16)) and np.array_equal(b.y, a.y.astype(np.float16))
    for name in ("s_in", "s_r", "s_out"):
        got, src = getattr(b, name), getattr(a, name)
        assert got.dtype == np.float32
        assert np.array_equal(got, src.astype(np.float16).astype(np.float32))
    assert np.array_equal(a.A_sign, b.A_sign) and np.array_equal(a.B_sign, b.B_sign)
    assert b.x_f64().dtype == np.float64 and np.array_equal(b.x_f64(), b.x.astype(np.float64))


def test_query_and_prepared_call_arguments_without_launching(lib):
    """lordba_query_variant, lordba_plan_bytes / _init / _launches and lordba_adapter_forward_planned
    reject bad arguments on the host; the independence check of a call is the same for all of them."""
    from paper_2605_24058_b200 import lordba
    EINVAL, EUNSUP, EALIGN = 1, 2, 3
    before = lordba.launch_count()
    one = (lordba.Proj * 1)(_proj(lordba))
    out = (ctypes.c_int * 4)()
    assert lib.lordba_query_variant(one, 1, 4, None, lordba.BF16, None) == EINVAL
    assert lib.lordba_query_variant(one, 1, -1, None, lordba.BF16, out) == EINVAL
    assert lib.lordba_query_variant(one, 1, 4, None, 9, out) == EUNSUP
    assert lib.lordba_query_variant(one, lordba.MAX_PROJS + 1, 4, None, lordba.BF16, out) == EUNSUP
    assert lib.lordba_query_variant(None, 0, 4, None, lordba.BF16, None) == 0
    # overlapping outputs; an input inside another projection's output; disjoint ones in any order
    two = (lordba.Proj * 2)(_proj(lordba), _proj(lordba, x=0x8000))
    assert lib.lordba_query_variant(two, 2, 4, None, lordba.BF16, out) == EINVAL
    chained = (lordba.Proj * 2)(_proj(lordba, x=0x300000, y=0x200000), _proj(lordba, x=0x200100, y=0x100000))
    assert lib.lordba_query_variant(chained, 2, 4, None, lordba.BF16, out) == EINVAL
    assert lib.lordba_plan_bytes(chained, 2, 4, None, lordba.BF16) == 0
    tok = (ctypes.c_int64 * 2)(4, 0)
    assert lib.lordba_query_variant(two, 2, 0, tok, lordba.BF16, out) in (0, 4)       # an empty segment overlaps nothing
    # float32 activations always run on the CUDA-core kernel: no device is needed to say so
    f32 = (lordba.Proj * 3)(_proj(lordba, y=0x100000), _proj(lordba, y=0x300000), _proj(lordba, y=0x200000))
    assert lib.lordba_query_variant(f32, 3, 4, None, lordba.F32, out) == 0
    assert [out[i] for i in range(3)] == [lordba.VARIANT_FMA] * 3
    # plans
    buf = (ctypes.c_char * 4096)()
    base = (ctypes.addressof(buf) + 63) // 64 * 64
    assert lib.lordba_plan_init(None, 1024, one, 1, 4, None, lordba.BF16) == EINVAL
    assert lib.lordba_plan_init(base + 8, 1024, one, 1, 4, None, lordba.BF16) == EALIGN
    assert lib.lordba_plan_init(base, 1024, two, 2, 4, None, lordba.BF16) == EINVAL
    assert lib.lordba_adapter_forward_planned(None, None) == EINVAL
    assert lib.lordba_adapter_forward_planned(base + 8, None) == EALIGN
    assert lib.lordba_adapter_forward_planned(base, None) == EINVAL          # zeros are not a plan
    assert lib.lordba_plan_launches(base) == -1 and lib.lordba_plan_launches(None) == -1
    assert lordba.launch_count() == before
