"""The C-ABI library loads and exports every symbol include/fdkv.h declares; host-side argument checks that
need no GPU (fdkv_sizes) behave."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = "".join(open(os.path.join(ROOT, "include", f)).read() for f in sorted(os.listdir(os.path.join(ROOT, "include")))
                   if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fdkv_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    from paper_2607_06519_b200 import build
    lib = C.CDLL(build.build())
    names = _declared()
    assert {"fdkv_compress_prefill", "fdkv_probe", "fdkv_decode_attn", "fdkv_kernel_launch_count", "fdkv_test_wait_expiry"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_sizes_and_config_validation():
    from paper_2607_06519_b200 import binding as B
    a, w = B.sizes(B.Config(32, 32, 8, 128, 1, 32768, 128, B.BF16, 1, 16))
    assert a >= 4 * 2 ** 30 and w >= 4 * 2 ** 30
    for bad in (B.Config(31, 32, 8, 128, 1, 1024, 8, B.BF16, 1, 16),    # odd layer count
                B.Config(32, 30, 8, 128, 1, 1024, 8, B.BF16, 1, 16),    # heads not divisible
                B.Config(32, 32, 8, 96, 1, 1024, 8, B.BF16, 1, 16),     # head_dim
                B.Config(32, 32, 8, 128, 1, 1 << 26, 8, B.BF16, 1, 16),  # flat index overflow
                B.Config(32, 32, 8, 128, 1, 1024, 8, 3, 1, 16),         # dtype
                B.Config(32, 32, 8, 128, 1, 1024, 8, B.BF16, 17, 16)):  # keep fraction > 1
        with pytest.raises(B.FdkvError):
            B.sizes(bad)


def test_no_gpu_means_loud_failure():
    import torch
    from paper_2607_06519_b200 import binding as B
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        B.Context(B.Config(2, 4, 2, 64, 1, 512, 1, B.F32, 1, 8))


def test_per_device_setup_table_runs_once_per_device():
    """Function attributes (the opt-in to large shared memory) belong to a device: the launchers' table must run its
    set-up on the first visit of EVERY device, not once per process."""
    from paper_2607_06519_b200 import build
    lib = C.CDLL(build.build())
    lib.fdkv_test_per_device_visits.restype = C.c_int32
    for devs, want in (([0, 0, 0], 1), ([0, 1, 0, 1, 2], 3), ([3], 1), ([], 0), ([0, 99, -1, 0], 1)):
        arr = (C.c_int32 * max(len(devs), 1))(*devs)
        assert lib.fdkv_test_per_device_visits(arr, len(devs)) == want, devs
