"""The C-ABI library loads without a GPU and exports every symbol that include/laq.h declares."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1909_07588_b200 import build, laq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return laq.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "laq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(laq_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(laq.EXPORTS) == names


def test_workspace_size_and_config_validation_need_no_gpu(lib):
    cfg, keep = laq.make_config(model=laq.MODEL_SYNTH, M=64, p=25_600_000, b=8)
    nbytes = laq.workspace_bytes(cfg)
    # Q_prev (M p fp32) + code streams (M p bytes) + theta and grad dominate
    assert 64 * 25_600_000 * 5 + 2 * 25_600_000 * 4 <= nbytes <= 64 * 25_600_000 * 5 + 2 * 25_600_000 * 4 + (8 << 20)
    for bad in (dict(b=5), dict(M=0), dict(D=0), dict(alpha=-1.0), dict(clock_mode=2), dict(p=0)):
        kw = dict(model=laq.MODEL_SYNTH, M=4, p=100, b=4)
        kw.update(bad)
        cfg, keep = laq.make_config(**kw)
        assert laq.workspace_bytes(cfg) == 0
    cfg, keep = laq.make_config(model=laq.MODEL_SOFTMAX, M=2, p=30, N=[5, 5], n_features=10, n_classes=4)
    assert laq.workspace_bytes(cfg) == 0            # p does not match C x F
    cfg, keep = laq.make_config(model=laq.MODEL_SOFTMAX, M=2, p=40, N=[5, 5], n_features=10, n_classes=4)
    assert laq.workspace_bytes(cfg) > 0


def test_struct_layout_matches_header(lib, tmp_path):
    """Compile the header as plain C and compare sizeof/offsetof with the ctypes mirrors."""
    import subprocess
    fields = {"laq_config": [f[0] for f in laq.laq_config._fields_],
              "laq_trace": [f[0] for f in laq.laq_trace._fields_],
              "laq_state": [f[0] for f in laq.laq_state._fields_]}
    c_name = lambda f: "lambda" if f == "lam" else f
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "laq.h"', 'int main(void){']
    for st, fs in fields.items():
        lines.append('printf("%s %%zu\\n", sizeof(%s));' % (st, st))
        for f in fs:
            lines.append('printf("%s.%s %%zu\\n", offsetof(%s, %s));' % (st, f, st, c_name(f)))
    lines.append("return 0;}")
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)],
                   check=True)
    out = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for st, fs in fields.items():
        cls = getattr(laq, st)
        assert ctypes.sizeof(cls) == int(out[st]), st
        for f in fs:
            assert getattr(cls, f).offset == int(out["%s.%s" % (st, f)]), (st, f)


def test_null_context_is_rejected(lib):
    assert lib.laq_step(None, 1, None) == laq.LAQ_EINVAL
    assert lib.laq_sync(None) == laq.LAQ_EINVAL
    assert lib.laq_last_error(None) == b"context is null"
    lib.laq_destroy(None)
