"""Host-only checks of the C ABI: the library builds for sm_100a, loads without a GPU, exports every
function the header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest
import torch

from paper_2604_04921_b200 import binding as tb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    tb.build()
    return tb.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "tri_attention.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tri_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(tb.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_layout_matches_header(lib, tmp_path):
    """Compile the header with gcc and compare sizeof/offsetof with the ctypes mirror."""
    import subprocess
    fields = {"tri_model_desc": [f for f, _ in tb._ModelDesc._fields_],
              "tri_cache_view": [f for f, _ in tb._CacheView._fields_]}
    src = ['#include <stdio.h>', '#include <stddef.h>', '#include "tri_attention.h"', 'int main(void){']
    for st, fs in fields.items():
        src.append(f'printf("{st} %zu\\n", sizeof({st}));')
        for f in fs:
            src.append(f'printf("{st}.{f} %zu\\n", offsetof({st}, {f}));')
    src.append('return 0;}')
    c = tmp_path / "layout.c"
    c.write_text("\n".join(src))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(c)], check=True)
    out = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for st, cls in (("tri_model_desc", tb._ModelDesc), ("tri_cache_view", tb._CacheView)):
        assert int(out[st]) == ctypes.sizeof(cls)
        for f, _ in cls._fields_:
            assert int(out[f"{st}.{f}"]) == getattr(cls, f).offset, (st, f)


def test_create_rejects_bad_descriptors(lib):
    qc = torch.zeros(1, 1, 128)
    qn = torch.zeros(1, 1, 64)
    with pytest.raises(tb.TriError) as e:
        tb.TriContext(1, 1, 1, torch.zeros(1, 1, 64), torch.zeros(1, 1, 32), head_dim=64)
    assert e.value.code == 2
    with pytest.raises(tb.TriError) as e:
        tb.TriContext(1, 1, 1, qc, qn, rope_theta=-1.0)
    assert e.value.code == 1
    with pytest.raises(tb.TriError) as e:
        tb.TriContext(1, 1, 1, qc, qn, offsets=[1, -2])
    assert e.value.code == 1
    with pytest.raises(tb.TriError) as e:
        tb.TriContext(1, 1, 1, qc, qn, norm_variant=7)
    assert e.value.code == 1
    with pytest.raises(tb.TriError) as e:
        tb.TriContext(1, 1, 17, torch.zeros(1, 17, 128), torch.zeros(1, 17, 64))
    assert e.value.code == 2


def test_null_arguments_are_rejected(lib):
    assert lib.tri_score(None, None, 1, None, None, None, None, 0, None) == 1
    assert lib.tri_select(None, None, None, 1, 1, 1, None, None, None, 0, None) == 1
    assert lib.tri_compact(None, None, None, None, 1, 1, None, None, None) == 1
    assert lib.tri_compress(None, None, 1, None, 1, None, None, None, None, None, None, 0, None) == 1
    assert lib.tri_workspace_bytes(None, 1, 1, 1) == 0
    assert lib.tri_destroy(None) == 0


def test_without_a_gpu_create_fails_loudly(lib):
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(tb.TriError) as e:
        tb.TriContext(1, 1, 1, torch.zeros(1, 1, 128), torch.zeros(1, 1, 64))
    assert e.value.code == 4
