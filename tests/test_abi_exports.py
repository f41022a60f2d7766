"""The shared library loads on a machine without a GPU and exports every
function that include/pb.h declares; no compute call is made here."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "pb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pb_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2003_11666_b200 import build
    build.build()
    import paper_2003_11666_b200 as p
    return p.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    import paper_2003_11666_b200 as p
    assert sorted(p.EXPORTS) == _declared()


def test_create_without_device_fails_with_status_not_crash(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("needs a machine without a GPU")
    import paper_2003_11666_b200 as p
    from pb_workloads import mlp
    wl = mlp([8, 4])
    with pytest.raises(p.PBError) as e:
        p.PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, 0.1, 0.9)
    assert e.value.code in (-3, -4)


def test_argument_checks_run_before_any_device_call(lib):
    import paper_2003_11666_b200 as p
    from pb_workloads import mlp, Layer, OP
    wl = mlp([8, 4])
    for bad in (dict(momentum=1.0), dict(lr=-1.0), dict(flags=64)):
        kw = dict(lr=0.1, momentum=0.9, flags=3)
        kw.update(bad)
        with pytest.raises(p.PBError) as e:
            p.PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, kw["lr"], kw["momentum"], kw["flags"])
        assert e.value.code == -1
    with pytest.raises(p.PBError) as e:      # layer list that does not chain
        p.PB(wl.layers, wl.stage_of_layer, (7, 1, 1), wl.n_classes, 0.1, 0.9)
    assert e.value.code == -2
    with pytest.raises(p.PBError) as e:      # stage without a head
        p.PB([Layer(OP.RELU)], [0], (3, 1, 1), 3, 0.1, 0.9)
    assert e.value.code == -1
