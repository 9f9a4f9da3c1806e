"""A plain C program drives one whole step of the path from pinned host memory (tests/c_step.c) and must
produce, bit for bit, what the Python binding's path produces on the same seeded batch."""
import os
import shutil
import subprocess

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _build_c_step(tmp_path):
    from paper_2401_13920_b200 import build
    lib = build.build()
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    exe = tmp_path / "c_step"
    subprocess.run([nvcc, "-O1", "-I", os.path.join(ROOT, "include"), os.path.join(ROOT, "tests", "c_step.c"), "-o", str(exe),
                    lib, "-Xlinker", "-rpath," + os.path.dirname(lib)], check=True)
    return exe


@pytest.mark.parametrize("cfg,T,cf,graph", [(2, 6000, 1.0, False), (5, 7001, 1.25, False), (2, 6000, 1.0, True), (5, 7001, 1.25, True)])
def test_c_program_step_equals_the_binding_path(tmp_path, cfg, T, cf, graph):
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2401_13920_b200 import binding as B
    from paper_2401_13920_b200 import workloads as W
    exe = _build_c_step(tmp_path)
    dev = torch.device("cuda:0")
    w = W.CONFIGS[cfg].scaled(T)
    x, src = W.make_tokens(w, dev), W.make_src(w, dev)
    W.host_bits(x).tofile(tmp_path / "x.bin")
    src.cpu().numpy().tofile(tmp_path / "src.bin")
    r = subprocess.run([str(exe), str(w.T), str(w.H), str(w.E), str(w.n_nodes), str(w.dev_per_node), repr(cf),
                        str(tmp_path / "x.bin"), str(tmp_path / "src.bin"), str(tmp_path / "out.bin"), str(tmp_path / "slot.bin")]
                       + (["graph"] if graph else []),
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.startswith("ok"), r.stdout + r.stderr
    sh = B.make_shape(w.T, w.H, w.E, w.n_nodes, w.dev_per_node, x.dtype)
    Ca = B.conventional_capacity(w.T, sh.D, w.E, cf)
    assert "C_alloc=%d " % Ca in r.stdout
    st = B.make_router(sh, Ca, B.CapacityRule(cf, cf, -1.0, 0, 0), dev)
    out = B.router_forward(st, x, src)
    torch.cuda.synchronize()
    assert np.array_equal(np.fromfile(tmp_path / "slot.bin", dtype=np.int32), st.slot.cpu().numpy())
    assert np.array_equal(np.fromfile(tmp_path / "out.bin", dtype=np.uint16).reshape(w.T, w.H), W.host_bits(out))
    assert 0 < int((st.slot < 0).sum()) < w.T
