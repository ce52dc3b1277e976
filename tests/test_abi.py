"""Host-side checks that need no GPU: the library loads, exports every function the header
declares, validates configurations before touching a device, and refuses to run without one."""
import ctypes
import re
from pathlib import Path

import pytest
import torch

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def binding():
    from paper_2408_15237_b200 import build
    build.build_library()
    from paper_2408_15237_b200 import binding as b
    return b


def declared_functions():
    text = (ROOT / "include" / "mamba_spec.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mamba_spec_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_three_named_entry_points():
    names = declared_functions()
    for want in ("mamba_spec_init", "mamba_spec_verify", "mamba_spec_commit"):
        assert want in names


def test_library_exports_every_declared_symbol(binding):
    names = declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(binding.lib, n), f"{n} is declared in include/mamba_spec.h but not exported"
        assert hasattr(binding, n), f"the Python binding lacks {n}"


def test_struct_layouts_match_the_header(binding):
    text = (ROOT / "include" / "mamba_spec.h").read_text()
    cfg = re.search(r"typedef struct \{([^{}]*)\} mamba_spec_config;", text).group(1)
    fields = re.findall(r"int32_t\s+(\w+);", cfg)
    assert fields == [f for f, _ in binding.Config._fields_]
    assert ctypes.sizeof(binding.Config) == 4 * len(fields)
    io = re.search(r"typedef struct \{([^{}]*)\} mamba_spec_io;", text).group(1)
    io = re.sub(r"/\*.*?\*/", "", io, flags=re.S)
    io_fields = re.findall(r"(\w+);", io)
    assert io_fields == [f for f, _ in binding.IO._fields_]


def cfg(binding, **over):
    base = dict(batch_max=2, n_layers=1, n_heads=8, head_dim=32, d_state=64, n_groups_b=2, n_groups_c=8,
                conv_width=4, k_max=4, act_dtype=binding.DTYPE_BF16, flags=3, device=0, kernel_select=0)
    base.update(over)
    return binding.Config(**base)


@pytest.mark.parametrize("over,code", [
    (dict(batch_max=0), -1), (dict(d_state=512), -4), (dict(conv_width=9), -4), (dict(n_groups_b=3), -2),
    (dict(k_max=33), -1), (dict(act_dtype=7), -1), (dict(flags=1 << 12), -1), (dict(flags=64), -1), (dict(kernel_select=5), -1),
    (dict(n_heads=1, head_dim=4, n_groups_b=1, n_groups_c=1), -2),
])
def test_init_rejects_bad_configurations_before_touching_a_device(binding, over, code):
    with pytest.raises(binding.MambaSpecError) as e:
        binding.mamba_spec_init(cfg(binding, **over))
    assert e.value.code == code
    assert "init:" in str(e.value)


def test_null_context_is_reported_not_dereferenced(binding):
    io = binding.IO()
    rc = binding.lib.mamba_spec_verify(None, None, None, None, None, None, None, None, None, None, 1, ctypes.byref(io))
    assert rc == binding.ERR_NOT_INIT
    assert binding.lib.mamba_spec_commit(None, None, 1, None) == binding.ERR_NOT_INIT
    assert binding.lib.mamba_spec_launch_count(None) == 0
    binding.lib.mamba_spec_destroy(None)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the behaviour on a machine without a GPU")
def test_no_cpu_fallback_init_fails_loudly_without_a_device(binding):
    with pytest.raises(binding.MambaSpecError) as e:
        binding.mamba_spec_init(cfg(binding))
    assert e.value.code == binding.ERR_CUDA
    assert "no CPU path" in str(e.value)


def test_product_package_never_imports_the_oracle():
    pkg = ROOT / "paper_2408_15237_b200"
    for f in list(pkg.rglob("*.py")) + list(pkg.rglob("*.cu")) + list(pkg.rglob("*.cuh")):
        assert not re.search(r"^\s*(import|from)\s+oracle\b|oracle/", f.read_text(), flags=re.M), f
    for f in (ROOT / "oracle").rglob("*"):
        if f.suffix in (".py", ".c", ".h"):
            assert "paper_2408_15237_b200" not in f.read_text(), f
