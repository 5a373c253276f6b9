"""The C-ABI library builds, loads without a GPU, and exports every function include/defl.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2609_21102_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "defl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(defl_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_two_primitives():
    names = _declared()
    assert "defl_polar_batched" in names and "defl_psd_project" in names
    assert len(names) >= 10


def test_library_exports_every_declared_symbol(libpath):
    L = ctypes.CDLL(libpath)
    for name in _declared():
        assert hasattr(L, name), name


def test_binding_lists_the_same_names(libpath):
    from paper_2609_21102_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    binding.lib()


def test_status_strings_and_no_device_behaviour(libpath):
    import torch
    L = ctypes.CDLL(libpath)
    L.defl_status_string.restype = ctypes.c_char_p
    for code in (0, -1, -2, -3, -4):
        assert len(L.defl_status_string(code)) > 0
    assert L.defl_polar_workspace_bytes(0, 4, 4, 0, 0, 0) == 0
    L.defl_polar_workspace_bytes.restype = ctypes.c_size_t
    assert L.defl_polar_workspace_bytes(2, 128, 256, 0, 4, 4) > 2 * 128 * 256 * 2
    if not torch.cuda.is_available():
        h = ctypes.c_void_p()
        # no CPU fallback: without a device the context cannot even be created
        assert L.defl_create(ctypes.byref(h), 0) == -3
        assert not h.value


def test_shape_groups_and_stacking():
    """Host-side grouping of a parameter list by stored shape (no GPU, no arithmetic)."""
    import torch
    from paper_2609_21102_b200 import grouping
    shapes = [(8, 4), (4, 8), (8, 4), (3,), (8, 4), (4, 8), (2, 2, 2)]
    g = grouping.shape_groups(shapes)
    assert list(g.items()) == [((8, 4), [0, 2, 4]), ((4, 8), [1, 5])]
    ts = [torch.full(s, float(i)) for i, s in enumerate(shapes)]
    buf, views = grouping.stack_group(ts, g[(8, 4)])
    assert buf.shape == (3, 8, 4) and [float(v[0, 0]) for v in views] == [0.0, 2.0, 4.0]
    views[1].add_(1.0)                      # a view writes through to the stacked buffer
    assert float(buf[1, 3, 3]) == 3.0
    with pytest.raises(ValueError):
        grouping.stack_group(ts, [0, 1])


def test_deflation_cutoff_switch():
    """Section 4, "Deflation cutoff": deflation during the first fraction of the optimizer steps, the plain step after;
    the step helper passes k = 0 past the cutoff (a recording stand-in for the context, no GPU)."""
    from paper_2609_21102_b200 import grouping
    assert [grouping.deflation_active(t, 10, 0.3) for t in range(10)] == [True] * 3 + [False] * 7
    assert all(grouping.deflation_active(t, 10, 1.0) for t in range(10))
    assert not any(grouping.deflation_active(t, 10, 0.0) for t in range(10))
    assert [grouping.deflation_active(t, 5, 0.5) for t in range(5)] == [True, True, True, False, False]   # 2.5 steps
    with pytest.raises(ValueError):
        grouping.deflation_active(0, 10, 1.5)

    class Recorder:
        def __init__(self):
            self.calls = []

        def defl_muon_step_batched(self, W, M, G, lr, mu, k, p, J, sched, **kw):
            self.calls.append((k, p, J))
    rec = Recorder()
    weights = {(1600, 6400): "W"}
    for t in range(4):
        grouping.muon_step_groups(rec, weights, {(1600, 6400): "M"}, {}, 0.02, 0.95, 0.02, 0.01, 2, [[1.0, 0.0, 0.0]],
                                  step=t, total_steps=4, cutoff=0.5)
    assert rec.calls == [(32, 16, 2), (32, 16, 2), (0, 16, 2), (0, 16, 2)]


def test_window_ratios_follow_the_algorithms(libpath):
    """Algorithm 3 line 1 (r = ceil(w m), r' = min{m, r + ceil(delta m)}) and Algorithm 2's inputs (r = ceil(w n),
    K = ceil(w' n)), worked by hand."""
    import pytest
    from paper_2609_21102_b200 import binding
    assert binding.defl_polar_window(1600, 6400, 0.02, 0.01) == (32, 16)
    assert binding.defl_polar_window(6400, 1600, 0.02, 0.01) == (32, 16)          # the short side counts
    assert binding.defl_polar_window(768, 3072, 0.01, 0.0105) == (8, 9)           # ceil(7.68) = 8, ceil(8.064) = 9
    assert binding.defl_polar_window(40, 40, 0.5, 0.9) == (20, 20)                # r' capped at the short side
    assert binding.defl_polar_window(40, 64, 1.0, 0.0) == (39, 0)                 # r capped at m - 1
    assert binding.defl_psd_window(4096, 8 / 4096, 16 / 4096) == (8, 16)
    assert binding.defl_psd_window(640, 0.025, 0.05) == (16, 32)
    with pytest.raises(binding.DeflError) as e:
        binding.defl_psd_window(5000, 0.025, 0.05)                                 # K = 250 exceeds the widest basis
    assert e.value.code == -2
    with pytest.raises(binding.DeflError) as e:
        binding.defl_polar_window(128, 256, -0.1, 0.0)
    assert e.value.code == -1
