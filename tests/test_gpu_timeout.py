"""The device-side timeout status, exercised without hanging or faulting anything.

Every barrier wait in the library's kernels is bounded: after its limit it records
SPARKATTN_E_DEVICE_TIMEOUT plus an id of the wait in the workspace's status words and the kernel
winds down.  The product kernels never meet that case on valid input, so this test builds a tiny
kernel of its own (tests/cuda/timeout_probe.cu) that calls the same `mbar_wait` helper on a barrier
nothing arrives at, with a limit of one millisecond, and reads the status back through the library's
sparkattn_read_status."""
import ctypes
import os
import subprocess
import time

import pytest
import torch

import paper_2609_23153_b200 as sa

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def probe(tmp_path_factory):
    out = str(tmp_path_factory.mktemp("probe") / "libtimeout_probe.so")
    src = os.path.join(HERE, "cuda", "timeout_probe.cu")
    subprocess.run(["nvcc", "-std=c++17", "-O2", "-gencode", "arch=compute_100a,code=sm_100a", "-shared",
                    "-Xcompiler", "-fPIC", "-o", out, src], check=True)
    lib = ctypes.CDLL(out)
    lib.timeout_probe.restype = ctypes.c_int
    lib.timeout_probe.argtypes = [ctypes.c_void_p, ctypes.c_ulonglong, ctypes.c_int, ctypes.c_void_p]
    return lib


def test_expired_wait_sets_timeout_status_and_returns(probe):
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda:0")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    t0 = time.perf_counter()
    assert probe.timeout_probe(ctypes.c_void_p(ws.data_ptr()), 1_000_000, 77, stream) == 0
    assert sa.read_status(ws) == sa.E_DEVICE_TIMEOUT          # synchronises: the kernel has returned
    elapsed = time.perf_counter() - t0
    words = ws.view(torch.int32).cpu()
    assert int(words[1]) == 77                                 # the id of the wait that gave up
    assert int(words[2]) == 32 and int(words[3]) == 0          # every thread left its wait unsuccessfully
    assert elapsed < 1.0, f"a 1 ms wait limit took {elapsed:.3f} s"
    # the context is still usable and a later library call on the same workspace starts clean
    x = torch.ones(1024, device="cuda:0")
    assert float(x.sum()) == 1024.0
