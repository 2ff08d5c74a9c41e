"""CPU-only checks of the boundary: the library loads without a GPU, exports every function that
include/decode_attn.h declares, and its host-side logic (status strings, options, argument
validation that runs before any CUDA call) behaves as documented."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "decode_attn.h")


@pytest.fixture(scope="module")
def pkg():
    from paper_2512_10977_b200 import build
    build.build()
    import paper_2512_10977_b200 as p
    return p


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(decode_attn\w*)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for want in ("decode_attn", "decode_attn_host_io", "decode_attn_workspace_bytes", "decode_attn_set_workspace",
                 "decode_attn_read_device_status", "decode_attn_plan", "decode_attn_strerror"):
        assert want in names


def test_library_loads_and_exports_every_declared_symbol(pkg):
    L = pkg.lib()
    for name in declared_functions():
        assert hasattr(L, name), f"{name} declared in the header but not exported"


def test_status_strings_and_version(pkg):
    L = pkg.lib()
    assert pkg.version() >= 100
    seen = {L.decode_attn_strerror(i).decode() for i in range(8)}
    assert len(seen) == 8 and all(seen)
    assert L.decode_attn_strerror(99).decode() == "unknown status"


def test_the_normal_build_keeps_no_timeline(pkg):
    # the stamps exist only in the -DDA_TIMELINE build; the normal library says so without touching CUDA
    buf = (ctypes.c_ulonglong * 16)()
    assert pkg.lib().decode_attn_timeline(buf, 16, 0) == 5   # DA_ERR_UNSUPPORTED
    with pytest.raises(pkg.DecodeAttnError):
        pkg.timeline()


def test_the_normal_build_knows_no_diagnostic_option(pkg):
    # shortening the kernels' wait limit or withholding a tile exists only in the diagnostic build
    for name in ("diag_wait_limit_us", "diag_withhold_partition_tile", "diag_withhold_prefix_tile"):
        assert pkg.lib().decode_attn_set_option(name.encode(), 1) == 5   # DA_ERR_UNSUPPORTED
        assert pkg.get_option(name) == -1


def test_options(pkg):
    assert pkg.get_option("grid_blocks") == 0
    pkg.set_option("grid_blocks", 7)
    assert pkg.get_option("grid_blocks") == 7
    pkg.set_option("grid_blocks", 0)
    with pytest.raises(pkg.DecodeAttnError) as e:
        pkg.set_option("grid_blocks", 10 ** 6)
    assert e.value.status == 5
    assert pkg.get_option("tail_units") == 4 and pkg.get_option("static_frac") == 224
    pkg.set_option("tail_units", 0)
    assert pkg.get_option("tail_units") == 0
    pkg.set_option("tail_units", 4)
    for name, bad in (("tail_units", 65), ("tail_units", -1), ("static_frac", 257)):
        with pytest.raises(pkg.DecodeAttnError) as e:
            pkg.set_option(name, bad)
        assert e.value.status == 5
    with pytest.raises(pkg.DecodeAttnError):
        pkg.set_option("no_such_option", 1)
    assert pkg.get_option("no_such_option") == -1


def test_workspace_size_grows_with_the_problem(pkg):
    a = pkg.workspace_bytes(1, 48, 8, 128, 16, 32)
    b = pkg.workspace_bytes(64, 48, 8, 128, 16, 1024)
    c = pkg.workspace_bytes(256, 48, 8, 128, 16, 2048)
    assert 0 < a < b < c
    assert pkg.workspace_bytes(-1, 48, 8, 128, 16, 32) == 0


def test_null_and_malformed_arguments_are_rejected_before_any_cuda_call(pkg):
    from paper_2512_10977_b200.binding import DaTensor
    L = pkg.lib()
    assert L.decode_attn(None, None, None, None, None, 0, 1.0, None, None, None) == 1

    def view(dtype, shape, data=0x1000):
        t = DaTensor()
        t.data, t.dtype, t.ndim = data, dtype, len(shape)
        stride = 1
        for i in reversed(range(len(shape))):
            t.shape[i], t.stride[i] = shape[i], stride
            stride *= shape[i]
        return t

    B, Hq, Hkv, P, D = 2, 48, 8, 16, 128
    q, k, v = view(1, (B, Hq, D)), view(1, (10, Hkv, P, D)), view(1, (10, Hkv, P, D))
    bt, sl, out, lse = view(3, (B, 4)), view(3, (B,)), view(2, (B, Hq, D)), view(2, (B, Hq))
    call = lambda *a: L.decode_attn(*[ctypes.byref(x) for x in a[:5]], 0, 1.0, ctypes.byref(a[5]), ctypes.byref(a[6]), None)
    assert call(view(2, (B, Hq, D)), k, v, bt, sl, out, lse) == 3                 # q must be bf16
    assert call(view(1, (B, 47, D)), k, v, bt, sl, view(2, (B, 47, D)), view(2, (B, 47))) == 2   # 47 % 8
    assert call(view(1, (B, Hq, 64)), k, v, bt, sl, out, lse) == 5                # head_dim
    assert call(q, view(1, (10, Hkv, 8, D)), view(1, (10, Hkv, 8, D)), bt, sl, out, lse) == 5    # page size
    assert call(q, view(1, (10, Hkv, P, D), data=0x1008), v, bt, sl, out, lse) == 4              # alignment
    assert call(q, k, view(1, (11, Hkv, P, D)), bt, sl, out, lse) == 2            # pools disagree
    assert call(view(1, (B, 8 * 17, D)), k, v, bt, sl, view(2, (B, 8 * 17, D)), view(2, (B, 8 * 17))) == 5  # group > 16
    assert call(q, k, v, view(3, (B + 1, 4)), sl, out, lse) == 2
    assert call(q, k, v, bt, sl, view(3, (B, Hq, D)), lse) == 3                   # out dtype
    null_q = view(1, (B, Hq, D), data=0)
    assert call(null_q, k, v, bt, sl, out, lse) == 1
    # pools without KV heads or without pages: a status, never a division fault on the host -- from the
    # single-token call and from the multi-token one (whose group size is Hq / Hkv)
    def pool(shape):
        t = view(1, shape)
        t.stride[0], t.stride[1], t.stride[2] = P * D * 8, P * D, D      # (zero extents must not make zero strides)
        return t
    q4, out4, lse3 = view(1, (B, 1, Hq, D)), view(2, (B, 1, Hq, D)), view(2, (B, 1, Hq))
    ext = lambda kk, vv: L.decode_attn_extend(ctypes.byref(q4), ctypes.byref(kk), ctypes.byref(vv), ctypes.byref(bt),
                                              ctypes.byref(sl), 1.0, ctypes.byref(out4), ctypes.byref(lse3), None)
    for shape in ((10, 0, P, D), (0, Hkv, P, D)):
        assert call(q, pool(shape), pool(shape), bt, sl, out, lse) == 2
        assert ext(pool(shape), pool(shape)) == 2
