"""The allocation-free thin-M entry point against the context's thin-M path (collected last on purpose).

gn_thin_m_gemm_noalloc serves callers that may not allocate device memory (a host application whose
allocator owns the whole GPU, a fixed memory budget, a latency-critical loop).  It runs the same kernels
as gn_debug_gemm(kind 2) on a [rows][M] x [rows][N] pair; only the scratch differs, so the two must agree
to the tolerance the other thin-kernel tests use - and, the chunking being identical, bit for bit.
"""
import numpy as np
import pytest

import gn_workloads as wl

pytestmark = pytest.mark.gpu


def test_two_calls_in_a_row_match_the_existing_entry_point():
    import torch
    import paper_1802_00130_b200 as gn
    p = wl.make("tiny")
    ctx = gn.GnContext(p["widths"], p["C"], torch.from_numpy(p["X"]).cuda(), torch.from_numpy(p["Y"]).cuda())
    rng = np.random.Generator(np.random.PCG64(2024))
    out = torch.empty((10, 2000), dtype=torch.float32, device="cuda")
    small = torch.empty((4, 64), dtype=torch.float32, device="cuda")
    # first call: the output layer's weight block at the headline network (|S| = 3000, n_L = 10, n_{L-1} = 2000);
    # second call: a much smaller problem, which must not pick up anything the first left in the shared scratch
    for (rows, M, N, dst) in ((3000, 10, 2000, out), (131, 4, 64, small), (3000, 10, 2000, out)):
        A = torch.from_numpy(rng.standard_normal((rows, M), dtype=np.float32)).cuda()
        B = torch.from_numpy(rng.standard_normal((rows, N), dtype=np.float32)).cuda()
        want = ctx.debug_gemm(2, A, B, a_kmajor=False, b_kmajor=False)
        dst.fill_(float("nan"))
        got = gn.thin_m_gemm_noalloc(A, B, dst)
        torch.cuda.synchronize()
        err = (got - want).norm().item() / want.norm().item()
        assert err <= 2e-6, err
        assert torch.equal(got, want)
        ref = A.double().t() @ B.double()
        assert ((got.double() - ref).norm() / ref.norm()).item() <= 2e-6
    ctx.close()


def test_sizes_beyond_the_built_in_scratch_are_refused_without_a_launch():
    import torch
    import paper_1802_00130_b200 as gn
    rows, M, N = 4096, 16, 4096          # 37 row chunks x 16 x 4096 floats > 2 097 152
    A = torch.zeros((rows, M), dtype=torch.float32, device="cuda")
    B = torch.zeros((rows, N), dtype=torch.float32, device="cuda")
    out = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(gn.GnError) as e:
        gn.thin_m_gemm_noalloc(A, B, out)
    assert e.value.status == 1 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())      # nothing ran
    with pytest.raises(gn.GnError) as e:  # M > 16 is not this kernel's shape
        gn.thin_m_gemm_noalloc(torch.zeros((64, 17), device="cuda"), torch.zeros((64, 64), device="cuda"),
                               torch.zeros((17, 64), device="cuda"))
    assert e.value.status == 1


_FIRST_CALL_SCRIPT = r"""
import sys
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
import paper_1802_00130_b200 as gn
rng = np.random.Generator(np.random.PCG64(7))
rows, M, N = 3000, 10, 2000
A = torch.from_numpy(rng.standard_normal((rows, M), dtype=np.float32)).cuda()
B = torch.from_numpy(rng.standard_normal((rows, N), dtype=np.float32)).cuda()
out = torch.empty((M, N), dtype=torch.float32, device="cuda")
ref = A.double().t() @ B.double()
side = torch.cuda.Stream()
torch.cuda.synchronize()
frees = []
for k in range(4):                      # the very first call into the library in this process is this entry point
    st = side if k == 2 else None       # once on a stream of the caller's own
    out.fill_(float("nan"))
    torch.cuda.synchronize()
    gn.thin_m_gemm_noalloc(A, B, out, stream=st)
    torch.cuda.synchronize()
    frees.append(torch.cuda.mem_get_info()[0])
    err = ((out.double() - ref).norm() / ref.norm()).item()
    assert err <= 2e-6, (k, err)
# the first call may make the runtime place the library's code and its fixed array on the device; from the second
# call on the device's free memory must not move by a byte
assert frees[1] == frees[2] == frees[3], frees
print("ok", frees)
"""


def test_first_library_call_in_a_fresh_process_and_no_byte_taken_afterwards():
    """A process whose first call into the library is this entry point (nothing else has made the runtime load the
    library's kernels), one call on a stream of the caller's own, and the device's free memory read after every
    call: identical from the second call on, which is what a caller whose allocator owns the rest of the memory
    relies on."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", _FIRST_CALL_SCRIPT, root], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.strip().startswith("ok")
