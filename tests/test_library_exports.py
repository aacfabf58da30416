"""The C-ABI library loads without a GPU and exports every symbol include/cosmoe.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2503_00245_b200 import build
    return ctypes.CDLL(build.build())


def declared():
    text = open(os.path.join(ROOT, "include", "cosmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in cosmoe.h but not exported"


def test_binding_covers_the_header():
    from paper_2503_00245_b200 import binding
    assert sorted(binding.EXPORTS) == declared()


def test_host_only_calls_work_without_a_gpu(lib):
    from paper_2503_00245_b200 import binding as B
    assert B._lib().moe_status_string(0) == b"ok"
    assert B._lib().moe_status_string(5) == b"a bounded wait expired"
    cfg = B.make_config(2048, 5632, 8, 2)
    assert B.moe_workspace_bytes(cfg, 1) > 2 * 5632 * 4
    assert B.moe_workspace_bytes(cfg, 2048) > 2048 * 2 * 2048 * 4
    for bad in (B.make_config(2047, 5632, 8, 2), B.make_config(2048, 5632, 8, 9), B.make_config(2048, 5632, 65, 2),
                B.make_config(2048, 5632, 2, 3)):
        with pytest.raises(B.MoeError) as e:
            B.moe_workspace_bytes(bad, 1)
        assert e.value.status == 2
    with pytest.raises(B.MoeError) as e:
        B.moe_workspace_bytes(B.make_config(0, 5632, 8, 2), 1)
    assert e.value.status == 1


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2503_00245_b200 import binding as B
    with pytest.raises(B.MoeError) as e:
        B.moe_create(B.make_config(256, 512, 8, 2))
    assert e.value.status in (4, 7)
