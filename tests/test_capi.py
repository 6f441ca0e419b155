"""The C ABI without a GPU: the library builds, loads and exports what include/iodf.h declares,
and descriptor validation (which is host-only) reports the documented status codes."""
import os
import re

import numpy as np
import pytest

import iodf_synth as S
import paper_2206_08869_b200 as G
from paper_2206_08869_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = G.load_library()
    header = open(os.path.join(ROOT, "include", "iodf.h")).read()
    declared = sorted(set(re.findall(r"\b(iodf_[a-z0-9_]+)\s*\(", header)))
    assert declared, "no declarations found"
    assert sorted(G.DECLARED_SYMBOLS) == declared
    for name in declared:
        assert hasattr(lib, name), name


def test_strerror():
    assert G.iodf_strerror(0) == "ok"
    for st in range(-8, 0):
        assert G.iodf_strerror(st) not in ("ok", "unknown status")
    assert G.iodf_strerror(-99) == "unknown status"


def _status(model, max_batch=4):
    try:
        G.iodf_create(model, max_batch)
    except G.IodfError as e:
        return e.status
    return 0


def _small():
    return S.make_model(5, 3, 8, 8, [True, False], 2, 12, prune=(0.4, 0.7))


def _no_device():
    try:
        import torch
        return not torch.cuda.is_available()
    except Exception:
        return True


def test_bad_descriptors_fail_on_the_host():
    EINVAL, ECUDA, EVERSION, EUNSUPPORTED, EOVERFLOW = -1, -3, -4, -6, -7
    m = _small()
    m["levels"][0]["couplings"][1]["perm"][:2] = 0
    assert _status(m) == EINVAL                      # not a permutation
    m = _small()
    m["levels"][0]["couplings"][0]["layers"][1]["m0"][0] = (1 << 30) - 1
    assert _status(m) == EINVAL                      # M0 below 2^30
    m = _small()
    m["levels"][1]["couplings"][0]["layers"][2]["s"][0] = 32
    assert _status(m) == EINVAL                      # shift out of range
    m = _small()
    m["levels"][0]["couplings"][0]["in_s"] = -1
    assert _status(m) == EINVAL
    m = _small()
    m["levels"][0]["couplings"][0]["layers"][0]["bias"][0] = 2**31 - 1
    assert _status(m) == EOVERFLOW                   # worst-case accumulator + bias
    m = _small()
    m["levels"][0]["couplings"][0]["layers"][2]["relu"] = True
    assert _status(m) == EINVAL                      # the translation layer must not clip
    m = _small()
    m["levels"][0]["couplings"][0]["layers"][0]["clamp"] = (-5, 300)
    assert _status(m) == EUNSUPPORTED                # after the ReLU 0..300: beyond the unsigned 8-bit range
    m = _small()
    m["levels"][0]["couplings"][0]["layers"][1]["clamp"] = (0, 256)
    assert _status(m) == EUNSUPPORTED
    m = _small()
    m["in_h"] = 6                                    # not divisible by 2^levels
    assert _status(m) == EINVAL
    assert _status(_small(), max_batch=0) == EINVAL
    # ABI version
    mm = binding._Marshalled(_small(), 4)
    mm.desc.abi_version = 99
    with pytest.raises(G.IodfError) as e:
        G.iodf_create(_small(), 4, marshalled=mm)
    assert e.value.status == EVERSION
    # a plan the library does not know
    mm = binding._Marshalled(_small(), 4, plan=7)
    with pytest.raises(G.IodfError) as e:
        G.iodf_create(_small(), 4, marshalled=mm)
    assert e.value.status == EINVAL
    # offsets beyond the blobs
    mm = binding._Marshalled(_small(), 4)
    mm.wts = mm.wts[:10].copy()
    with pytest.raises(G.IodfError) as e:
        G.iodf_create(_small(), 4, marshalled=mm)
    assert e.value.status == EINVAL
    if _no_device():
        assert _status(_small()) == ECUDA            # valid model, but no device to put it on


def test_gated_models_must_be_compacted():
    dense = S.masked_dense_model(_small(), 9, 12)
    with pytest.raises(ValueError):
        G.iodf_create(dense, 4)


def test_residual_couplings_beyond_the_kernels_limits_are_refused():
    """Residual-block couplings run for levels of at most 2048 pixels per image (eight row bands of
    256 pixels) and widths up to 128; anything else must be refused on the host (IODF_EUNSUPPORTED),
    a malformed index list is EINVAL."""
    m = S.make_residual_model(3, 3, 128, 128, [True], 1, 8, 1)        # 4096 pixels at the level
    assert _status(m) == -6
    m = S.make_residual_model(3, 3, 2, 1024, [True], 1, 8, 1)         # one row of 512 pixels: no bands of two rows
    assert _status(m) == -6
    m = S.make_residual_model(3, 3, 8, 8, [True], 1, 136, 1)          # hidden width above 128
    assert _status(m) == -6
    m = S.make_residual_model(3, 3, 8, 8, [True], 1, 8, 1)
    m["levels"][0]["couplings"][0]["blocks"][0]["idx"][:] = 0
    assert _status(m) == -1
