"""Host-side checks of the C ABI that need no GPU: the library builds and loads,
exports every symbol the header declares, the header is valid C99 and its
structs have the layout the ctypes binding assumes, and without a CUDA device
the library refuses to work (there is no CPU path)."""
import ctypes as C
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "muloco.h")


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as g
    g.build()
    from paper_2505_23725_b200 import binding
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    from paper_2505_23725_b200 import binding
    text = open(HEADER).read()
    declared = sorted(set(re.findall(r"MULOCO_API[^;(]*?\b(muloco_[a-z_]+)\s*\(", text)))
    assert len(declared) >= 16
    assert sorted(binding.EXPORTS) == declared
    for name in declared:
        assert getattr(lib, name) is not None


def test_header_is_c99_and_struct_layout_matches_binding(tmp_path):
    from paper_2505_23725_b200 import binding
    src = tmp_path / "t.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "muloco.h"\n'
                   'int main(void){printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(muloco_config), sizeof(muloco_tensor_desc),'
                   ' sizeof(muloco_buffers), offsetof(muloco_config, workspace_bytes), offsetof(muloco_config, outer_lr),'
                   ' offsetof(muloco_tensor_desc, wd_mult)); return 0;}\n')
    exe = tmp_path / "t"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    out = subprocess.check_output([str(exe)]).decode().split()
    assert [int(x) for x in out] == [C.sizeof(binding.Config), C.sizeof(binding.TensorDesc), C.sizeof(binding.Buffers),
                                     binding.Config.workspace_bytes.offset, binding.Config.outer_lr.offset,
                                     binding.TensorDesc.wd_mult.offset]


def test_create_validates_and_has_no_cpu_path(lib):
    from paper_2505_23725_b200 import binding, configs
    import torch
    w = configs.mini_workload()
    cfg = binding.make_config(w)
    ctx = C.c_void_p()
    # bad configuration: J does not divide H -- rejected before any device work
    bad = binding.make_config(w, H=4, J=3)
    assert lib.muloco_create(C.byref(bad), None, 0, None, None, C.byref(ctx)) == binding.EINVAL
    assert b"divide" in lib.muloco_last_error(None)
    bad = binding.make_config(w, K=0)
    assert lib.muloco_create(C.byref(bad), None, 0, None, None, C.byref(ctx)) == binding.EINVAL
    bad = binding.make_config(w, quant=3)
    assert lib.muloco_create(C.byref(bad), None, 0, None, None, C.byref(ctx)) == binding.EINVAL
    st = lib.muloco_create(C.byref(cfg), None, 0, None, None, C.byref(ctx))
    if torch.cuda.is_available():
        assert st == binding.OK
        lib.muloco_destroy(ctx)
    else:
        assert st == binding.ECUDA and not ctx.value
        assert b"no CPU path" in lib.muloco_last_error(None)
        with pytest.raises(RuntimeError):
            binding.MuLoCo(w)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_23725_b200")
    imp = re.compile(r"^\s*(from|import)\s+oracle\b|#include\s+[\"<].*oracle", re.M)
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert not imp.search(open(os.path.join(dirpath, f)).read()), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2505_23725_b200" not in text and "ctypes" not in text


def test_cosine_schedule_endpoints_midpoint_and_monotonicity():
    """Section 5: cosine decay to 0.1x the maximum.  Closed-form points of the half cosine."""
    from paper_2505_23725_b200.configs import cosine_lr_scale as f
    T, W = 1001, 100
    assert f(0, T) == 1.0 and abs(f(T - 1, T) - 0.1) < 1e-15
    assert abs(f(500, T) - 0.55) < 1e-12                      # midpoint: (1 + 0.1) / 2
    assert abs(f(250, T) - (0.1 + 0.9 * 0.5 * (1 + 2 ** -0.5))) < 1e-12   # quarter: cos(pi/4)
    assert f(0, T, W) == 1 / W and f(W - 1, T, W) == 1.0 and f(W, T, W) == 1.0
    xs = [f(t, T, W) for t in range(W, T)]
    assert all(a >= b for a, b in zip(xs, xs[1:])) and abs(xs[-1] - 0.1) < 1e-15
    assert f(5 * T, T) == pytest.approx(0.1)                  # past the end: stays at the floor
    with pytest.raises(ValueError):
        f(0, 0)
    with pytest.raises(ValueError):
        f(0, 10, 10)
