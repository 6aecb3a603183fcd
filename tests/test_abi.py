"""CPU-side checks of the boundary: the library loads, exports every function include/moe.h declares,
and its pure-host entry points behave.  No compute call is made (there may be no GPU)."""
import ctypes as C
import os
import re

import pytest

from paper_2607_23264_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text)))


def test_header_functions_are_exported(lib):
    names = declared_functions()
    assert "moe_fused_forward" in names and "moe_plan_routing" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/moe.h but not exported"
    assert sorted(binding.EXPORTS) == names, "binding.EXPORTS out of step with the header"


def test_status_strings(lib):
    assert binding.moe_status_string(0) == "MOE_OK"
    assert binding.moe_status_string(6) == "MOE_ERR_TIMEOUT"
    for code, name in binding.STATUS_NAMES.items():
        assert binding.moe_status_string(code) == name
    assert binding.moe_status_string(99) == "MOE_ERR_UNKNOWN"


def test_workspace_layout_is_aligned_and_ordered(lib):
    T, H, F, E, k = 128, 256, 512, 8, 2
    L = binding.moe_get_workspace_layout(T, H, F, E, k)
    assert L["total"] == binding.moe_workspace_bytes(T, H, F, E, k)
    R = T * k
    sizes = dict(topk_ids=R * 4, topk_w=R * 4, counts=E * 4, offsets=(E + 1) * 4, perm=R * 4, inv_perm=R * 4,
                 x_perm=R * H * 2, h=R * F * 2, y_perm=R * H * 2, x_stage=T * H * 2, logits_stage=T * E * 4,
                 out_stage=T * H * 2, x_stage_b=T * H * 2, logits_stage_b=T * E * 4, out_stage_b=T * H * 2)
    prev_end = 0
    for name, size in sizes.items():
        assert L[name] % 256 == 0
        assert L[name] >= prev_end, f"{name} overlaps its predecessor"
        prev_end = L[name] + size
    assert L["total"] >= prev_end


@pytest.mark.parametrize("shape", [
    (8, 100, 128, 4, 2),     # H not a multiple of 64
    (8, 128, 96, 4, 2),      # F not a multiple of 64
    (8, 128, 128, 4, 5),     # k > E
    (8, 128, 128, 2048, 2),  # E too large
    (8, 128, 128, 64, 33),   # k > 32
    (-1, 128, 128, 4, 2),    # T < 0
])
def test_bad_shapes_are_rejected_on_the_host(lib, shape):
    assert binding.moe_workspace_bytes(*shape) == 0
    with pytest.raises(binding.MoeError) as ei:
        binding.moe_get_workspace_layout(*shape)
    assert ei.value.code == 2


def test_ep_size_other_than_one_is_unsupported(lib):
    s = binding.moe_shape(8, 128, 128, 4, 2, 2, 0)
    out = binding.moe_workspace_layout()
    assert lib.moe_get_workspace_layout(C.byref(s), C.byref(out)) == 7
    assert lib.moe_workspace_bytes(C.byref(s)) == 0


def test_null_arguments(lib):
    assert lib.moe_get_workspace_layout(None, None) == 1
    assert lib.moe_create(None, None, 0) == 1
    lib.moe_destroy(None)
    assert lib.moe_last_launch_count(None) == 0
    assert lib.moe_plan_routing(None, None, None, None, None, None, None, None, None) == 1


def test_tuning_string_parser(lib):
    """The parser behind the MOE_TUNING environment override (pure host code)."""
    t, named = binding.moe_parse_tuning(None)
    assert not named and (t.store_burst_tiles, t.interleave_mode, t.interleave_k, t.schedule, t.dep_lead_D,
                          t.debug_flags) == (1, 0, 1, 0, 0, 0)
    t, named = binding.moe_parse_tuning("burst=4,mode=1,k=2")
    assert named and (t.store_burst_tiles, t.interleave_mode, t.interleave_k) == (4, 1, 2) and t.schedule == 0
    t, named = binding.moe_parse_tuning("schedule=1, lead=8,flags=0x1")
    assert named and (t.schedule, t.dep_lead_D, t.debug_flags) == (1, 8, 1)
    t, named = binding.moe_parse_tuning("x.some_knob=3")
    assert not named, "development knobs alone do not replace the default tuning"
    for bad in ("burst=3", "bogus=1", "burst", "burst=", "k=1x", "lead=4", "mode=2", "=1"):
        with pytest.raises(binding.MoeError) as ei:     # lead without schedule 1, values moe_tuning does not allow
            binding.moe_parse_tuning(bad)
        assert ei.value.code == 1, bad


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()
