"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its host-side
validation rejects bad requests before anything would be launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ebs():
    import paper_2003_07577_b200 as pkg
    pkg.build()
    return pkg.binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ebs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ebs_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(ebs):
    L = ebs.lib()
    names = declared_functions()
    assert len(names) >= 14
    for name in names:
        assert hasattr(L, name), f"{name} declared in ebs.h but not exported"
    assert sorted(ebs.EXPORTS) == names
    for name in names:                                  # the binding mirrors every entry point
        if name not in ("ebs_last_cuda_error", "ebs_conv2d_mixed_variant"):
            assert hasattr(ebs, name), name


def test_sizes_and_shapes(ebs):
    d = ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 2, 2, 0.05, 0.05)
    assert ebs.ebs_packed_weight_plane_bytes(d) == 3 * 3 * 2 * 64 * 2 * 4   # same bits as the unpacked weights
    assert ebs.ebs_packed_weight_plane_bytes(d) * 8 == 64 * 64 * 9 * 2
    assert ebs.ebs_packed_weight_bytes(d) == 3 * 3 * 2 * 64 * 2 * 4 + 3 * 3 * 2 * 64 * 32   # + one byte per weight
    d5 = ebs.conv_desc(3, 5, 1, 1, 1, 1, 0, 0, 3, 2, 0.05, 0.05)
    assert ebs.ebs_packed_weight_plane_bytes(d5) == 256 and ebs.ebs_packed_weight_bytes(d5) == 256 + 16 * 32
    assert ebs.ebs_packed_act_bytes(1, 32, 32, 64, 2) == 32 * 32 * 2 * 2 * 4
    assert ebs.ebs_packed_act_bytes(2, 5, 5, 33, 3) == 2 * 25 * 2 * 3 * 4
    assert ebs.ebs_conv_out_shape(d, 32, 32) == (32, 32)
    d2 = ebs.conv_desc(3, 64, 7, 7, 2, 2, 3, 3, 8, 8, 0.05, 0.05)
    assert ebs.ebs_conv_out_shape(d2, 224, 224) == (112, 112)
    assert ebs.ebs_version() >= 100 and ebs.ebs_num_conv_variants() == 41
    assert ebs.ebs_status_string(0) == "ok" and "overflow" in ebs.ebs_status_string(-3)
    assert ebs.ebs_host_workspace_bytes(d, 1, 32, 32, ebs.EBS_U8_CODES, 2) >= 65536 + 16384 + 2 * 262144 + 16384


def test_validation_rejects_bad_requests_without_launching(ebs):
    L = ebs.lib()
    good = ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 2, 2, 0.05, 0.05)
    fake = ctypes.c_void_p(0x1000)                        # aligned, never dereferenced: validation fails first
    ref = ctypes.byref

    def conv(desc, n=1, h=8, w=8, x=fake, wt=fake, acc=fake, y=None, pn=None, epi=None):
        return L.ebs_conv2d_mixed(x, n, h, w, wt, ref(desc), epi, acc, y, pn, None)

    assert conv(ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 9, 2, 0.05, 0.05)) == ebs.EBS_ERR_INVALID_ARG
    assert conv(ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 2, 0, 0.05, 0.05)) == ebs.EBS_ERR_INVALID_ARG
    assert conv(ebs.conv_desc(0, 64, 3, 3, 1, 1, 1, 1, 2, 2, 0.05, 0.05)) == ebs.EBS_ERR_INVALID_ARG
    assert conv(ebs.conv_desc(64, 64, 3, 3, 0, 1, 1, 1, 2, 2, 0.05, 0.05)) == ebs.EBS_ERR_INVALID_ARG
    assert conv(ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 2, 2, -1.0, 0.05)) == ebs.EBS_ERR_INVALID_ARG
    assert conv(good, x=None) == ebs.EBS_ERR_INVALID_ARG
    assert conv(good, acc=None) == ebs.EBS_ERR_INVALID_ARG                 # no output requested
    assert conv(good, acc=ctypes.c_void_p(0x1004)) == ebs.EBS_ERR_INVALID_ARG   # misaligned
    assert conv(good, n=0) == ebs.EBS_ERR_INVALID_ARG
    assert conv(ebs.conv_desc(64, 64, 9, 9, 1, 1, 0, 0, 2, 2, 0.05, 0.05), h=4, w=4) == ebs.EBS_ERR_INVALID_ARG
    assert conv(good, pn=fake) == ebs.EBS_ERR_INVALID_ARG                  # packed output needs an epilogue
    # 8-bit x 8-bit over 70 000 reduction elements cannot be held in int32
    assert conv(ebs.conv_desc(70000, 8, 1, 1, 1, 1, 0, 0, 8, 8, 0.05, 0.05)) == ebs.EBS_ERR_OVERFLOW
    assert ebs.ebs_packed_weight_bytes(ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 2, 12, 0.05, 0.05)) == 0
    assert L.ebs_pack_acts(fake, 7, 0, 1, 3, 4, 4, 2, 0.1, fake, None) == ebs.EBS_ERR_INVALID_ARG
    assert L.ebs_pack_acts(fake, ebs.EBS_F32, 0, 1, 3, 4, 4, 2, 0.0, fake, None) == ebs.EBS_ERR_INVALID_ARG
    assert L.ebs_pack_weights(None, ebs.EBS_I8_CODES, 0, ref(good), fake, None) == ebs.EBS_ERR_INVALID_ARG
    assert L.ebs_dequant(fake, 0, 4, 1.0, None, None, 0, fake, None) == ebs.EBS_ERR_INVALID_ARG
    assert L.ebs_probe_pipe(9, 10, ref(ctypes.c_double())) == ebs.EBS_ERR_INVALID_ARG
    with pytest.raises(ebs.EbsError):
        ebs.ebs_conv_out_shape(ebs.conv_desc(64, 64, 9, 9, 1, 1, 0, 0, 2, 2, 0.05, 0.05), 4, 4)


def test_product_package_does_not_touch_the_oracle():
    pkg_dir = os.path.join(ROOT, "paper_2003_07577_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2003_07577_b200" not in text and "ebs.h" not in text
