"""Host-side checks of the C ABI: the library loads, exports every symbol the header declares,
and its host-only helpers agree with the oracle's definition of the packed layout."""
import os
import re

import numpy as np
import pytest

import oracle
import paper_2002_11082_b200 as ogq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ogq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ogq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    for required in ("ogq_levels_bingrad", "ogq_levels_orq", "ogq_quantize_pack", "ogq_unpack_sum",
                     "ogq_workspace_bytes", "ogq_packed_layout"):
        assert required in names
    L = ogq.lib()
    for n in names:
        assert hasattr(L, n), n


def test_binding_has_the_same_names():
    for n in declared_functions():
        assert hasattr(ogq, n), n


def test_bits_and_layout_match_the_oracle_format():
    assert [ogq.ogq_bits_for_levels(s) for s in (2, 3, 5, 9, 17, 1, 33)] == [1, 2, 3, 4, 5, 0, 0]
    for s in (2, 3, 5, 9, 17):
        assert ogq.ogq_bits_for_levels(s) == oracle.bits_for(s)
    off = np.array([0, 0, 1, 33, 160, 160, 4257, 70000], np.int64)
    for bits in range(1, 6):
        assert np.array_equal(ogq.ogq_packed_layout(off, bits), oracle.packed_layout(off, bits))
    with pytest.raises(ogq.OgqError):
        ogq.ogq_packed_layout(off, 6)
    with pytest.raises(ogq.OgqError):
        ogq.ogq_packed_layout(np.array([0, 5, 3], np.int64), 2)


def test_workspace_bytes_is_monotone_and_positive():
    a = ogq.ogq_workspace_bytes(1, 1 << 16, 3)
    b = ogq.ogq_workspace_bytes(161, 25557032, 17)
    assert 0 < a <= b
    assert ogq.ogq_workspace_bytes(-1, 5, 3) == 0


def test_selection_solvers_refuse_buckets_of_2_to_the_32_elements():
    """The ORQ and BinGrad-pb solvers count in 32-bit cells: the header gives the limit and the call
    returns OGQ_ERR_UNSUPPORTED before it touches the device (no GPU needed for this check)."""
    big = 1 << 32
    dummy = 256  # never dereferenced: the size check comes first
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_orq(dummy, dummy, 1, big, 9, dummy, dummy, dummy, 1 << 40, stream=0)
    assert e.value.code == 2
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_bingrad(dummy, dummy, 1, big, ogq.OGQ_BINGRAD_PB, 0, dummy, dummy, dummy, dummy, 1 << 40,
                               stream=0)
    assert e.value.code == 2


def test_workspace_of_the_vgg19_bucket_is_a_fraction_of_the_gradient():
    """The key buffers hold one eighth of the bucket each (copies that do not fit make the solver read
    the gradient again): 143.7 M elements need well under 0.3 GB of scratch."""
    ws = ogq.ogq_workspace_bytes(38, 143667240, 17)
    assert ws < 0.3e9
    assert ws < 1.2 * 143667240 + 38 * 100_000
