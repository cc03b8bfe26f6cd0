"""The bounded barrier wait of the tensor-core kernels, made to run out on purpose.

A test-only kernel (tests/cuda/wait_timeout.cu, compiled here with nvcc) waits with a limit of a few thousand
cycles on an mbarrier that nothing arrives on: the wait returns false, marks the waiter dead, counts one failure
per waiting thread, later waits return at once and the kernel ends with the context intact.  The library's own
kernels must report no such failure.
"""
import ctypes as C
import os
import subprocess

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def probe(tmp_path_factory):
    out = str(tmp_path_factory.mktemp("wait") / "libwait_timeout.so")
    nvcc = "/usr/local/cuda/bin/nvcc" if os.path.exists("/usr/local/cuda/bin/nvcc") else "nvcc"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-std=c++17", "-shared", "-Xcompiler", "-fPIC",
           "-cudart", "static", "-I", os.path.join(ROOT, "paper_1804_02941_b200", "csrc"), "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "cuda", "wait_timeout.cu"), "-o", out]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    lib = C.CDLL(out)
    lib.run_wait_timeout.argtypes = [C.c_longlong, C.c_int, C.c_void_p, C.c_void_p]
    lib.run_wait_timeout.restype = C.c_int
    return lib


@pytest.mark.parametrize("threads", [1, 32, 96])
def test_a_wait_that_nothing_ends_runs_out_and_is_counted(probe, threads):
    torch.cuda.init()
    failures = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    rc = probe.run_wait_timeout(20000, threads, C.c_void_p(failures.data_ptr()), C.c_void_p(out.data_ptr()))
    assert rc == 0                                         # the kernel ended, the context is usable
    assert out.cpu().tolist() == [0, 0, 1, 1]              # both waits failed, the first only after the limit
    assert int(failures.item()) == threads                 # one count per waiting thread, none for the second wait
    assert float((torch.ones(8, device="cuda") * 2).sum().item()) == 16.0


def test_the_library_kernels_report_no_wait_that_ran_out():
    import paper_1804_02941_b200 as d
    d.lib()
    assert d.dab_contraction_wait_failures() == 0
