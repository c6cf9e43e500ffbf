"""A bounded device-side wait that runs out: the kernel records it and returns, the
host reads FO_ERR_DEVICE_TIMEOUT, the workspace is cleared and usable again.

Nothing faults or hangs: the test kernel (compiled here, not part of the library)
waits a few polls on a shared-memory barrier that nobody arrives at and that no
copy targets, sets the status word the library's kernels set in that situation,
and exits with nothing in flight."""
import ctypes as C
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_1801_00829_b200", "csrc")

SOURCE = r"""
#include "common.cuh"
#include "ptx.cuh"

__global__ void wait_for_nobody(fo::WsHead *head, unsigned polls)
{
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        fo::mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // phase 0 of `bar` completes only after an arrival that never comes
    const bool done = fo::mbar_wait(&bar, 0u, polls);
    if (!done && threadIdx.x == 0) atomicExch(&head->status, 1u);
}

extern "C" int launch_wait_for_nobody(void *ws, unsigned polls, void *stream)
{
    wait_for_nobody<<<1, 32, 0, (cudaStream_t)stream>>>((fo::WsHead *)ws, polls);
    return (int)cudaGetLastError();
}
"""


def test_a_wait_that_runs_out_is_reported_and_cleared(tmp_path):
    import torch
    import paper_1801_00829_b200 as fo
    from paper_1801_00829_b200 import binding as B
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc) and shutil.which("nvcc") is None:
        pytest.skip("no nvcc to build the test kernel with")
    src = tmp_path / "wait_for_nobody.cu"
    src.write_text(SOURCE)
    lib_path = tmp_path / "libwait.so"
    subprocess.run([nvcc, "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-gencode",
                    "arch=compute_100a,code=sm_100a", "-I", CSRC, "-I", os.path.join(ROOT, "include"),
                    "-o", str(lib_path), str(src)], check=True, capture_output=True)
    test_lib = C.CDLL(str(lib_path))
    test_lib.launch_wait_for_nobody.argtypes = [C.c_void_p, C.c_uint, C.c_void_p]
    test_lib.launch_wait_for_nobody.restype = C.c_int

    lib = fo.load_library()
    dev = torch.device("cuda", 0)
    ws = fo.workspace(dev, 16384)
    assert fo.device_status(dev) == 0
    assert test_lib.launch_wait_for_nobody(C.c_void_p(ws.data_ptr()), 8, None) == 0
    torch.cuda.synchronize()
    assert fo.device_status(dev) == -7                         # FO_ERR_DEVICE_TIMEOUT
    assert lib.fo_status_string(-7).decode() == "a bounded device-side wait ran out"
    # the context is intact: clear the control words and carry on
    assert lib.fo_workspace_init(C.c_void_p(ws.data_ptr()), ws.numel(), B._stream(dev)) == 0
    assert fo.device_status(dev) == 0
    X = torch.ones((300, 200), dtype=torch.float64, device=dev)
    assert fo.fused_cell([("sq", "t0", "a")], "t0", X).item() == 60000.0
    assert fo.device_status(dev) == 0
