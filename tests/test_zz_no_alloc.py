"""The allocation-free logsumexp entry point, mtmc_linear_lse_noalloc.

Some callers of this library are not allowed to allocate device memory: an operator
running inside a serving loop (a cudaMalloc there stalls the whole device), a plug-in
inside a framework whose own pool already holds the GPU.  For them the library keeps
the logsumexp partials in an 8 MiB array built into its image.  The tests call the
entry point through the C ABI twice in a row -- the second call finds the first
call's leftovers in the shared array -- and check both results against the fp64
oracle and against the regular mtmc_linear_lse, within the fp32 tolerance used
throughout (1e-3 + 1e-3 |ref|).  A child process, in which this entry point is the
only thing the library is ever asked to do, checks the property the entry point
exists for: the library's own count of device allocations stays at zero and the
device's free memory does not move.

Nothing here depends on what ran before in the process: the tests pass alone in a
fresh interpreter (where theirs is the first call the library sees) and after the
rest of the suite."""
import os
import subprocess
import sys

import pytest
import torch

from oracle import ref
from paper_2511_20100_b200 import binding as B
from paper_2511_20100_b200 import inputs

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _within(a: torch.Tensor, want: torch.Tensor) -> bool:
    a, want = a.double(), want.double()
    return bool((torch.isfinite(a)).all()) and bool(((a - want).abs() <= 1e-3 + 1e-3 * want.abs()).all())


def test_noalloc_matches_oracle_and_regular_entry_point_twice_in_a_row():
    first = inputs.linear_inputs(300, 3000, 256, seed=71)        # several column tiles, ragged M and N
    second = inputs.linear_inputs(200, 520, 448, seed=72)        # different shape: stale partials must not leak in
    for li in (first, second):
        Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
        M = Xd.shape[0]
        got = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
        mem_before = torch.cuda.memory_allocated()
        allocs_before = B.mtmc_device_alloc_count()
        B.mtmc_linear_lse_noalloc(Xd, Wd, bd, got)
        assert torch.cuda.memory_allocated() == mem_before      # the binding allocated no tensor either
        assert B.mtmc_device_alloc_count() == allocs_before     # and the library made no cudaMalloc
        torch.cuda.synchronize()
        oracle = ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b))
        r = ref.compare(inputs.to_f64(got), oracle, 1e-3, 1e-3)
        assert r["ok"], "against the oracle: %r" % (r,)
        want = B.mtmc_linear_lse(Xd, Wd, bd)
        B.mtmc_check_status()
        assert _within(got, want), "max |diff| %.3e" % float((got - want).abs().max())


def test_noalloc_without_bias_and_repeatable():
    li = inputs.linear_inputs(129, 1000, 128, seed=73, bias=False)
    Xd, Wd = li.X.cuda(), li.W.cuda()
    a = torch.empty(129, dtype=torch.float32, device="cuda")
    b = torch.empty(129, dtype=torch.float32, device="cuda")
    B.mtmc_linear_lse_noalloc(Xd, Wd, None, a)
    B.mtmc_linear_lse_noalloc(Xd, Wd, None, b)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    assert _within(a, B.mtmc_linear_lse(Xd, Wd, None))
    r = ref.compare(inputs.to_f64(a), ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), None), 1e-3, 1e-3)
    assert r["ok"], "against the oracle: %r" % (r,)


def test_noalloc_rejects_shapes_beyond_its_scratch():
    # ceil(N/256) * M = 4 * 300000 = 1,200,000 > 1,048,576: refused before anything is enqueued.
    L = B.load()
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(64, dtype=torch.float32, device="cuda")
    before = B.mtmc_launch_count()
    rc = L.mtmc_linear_lse_noalloc(x.data_ptr(), x.data_ptr(), None, 300000, 1024, 64, o.data_ptr())
    assert rc == B.ERR_UNSUPPORTED_SHAPE
    assert b"mtmc_linear_lse" in L.mtmc_last_error()
    assert B.mtmc_launch_count() == before


_CHILD = r"""
import sys
sys.path.insert(0, %r)
import torch
from paper_2511_20100_b200 import binding as B
from paper_2511_20100_b200 import inputs
torch.cuda.set_device(0)
small = inputs.linear_inputs(64, 256, 64, seed=1)
mid = inputs.linear_inputs(1024, 8192, 512, seed=2)
big = inputs.linear_inputs(4096, 32000, 256, seed=3)          # the LM-head shape's M and N: 512,000 of the 1,048,576 partials
dev = [(t.X.cuda(), t.W.cuda(), t.b.cuda(), torch.empty(t.X.shape[0], dtype=torch.float32, device="cuda")) for t in (small, mid, big)]
B.load()
torch.cuda.synchronize()
B.mtmc_linear_lse_noalloc(*dev[0])        # first call: one-time set-up (module load, symbol address)
torch.cuda.synchronize()
free0 = torch.cuda.mem_get_info()[0]
for _ in range(2):
    for d in dev:
        B.mtmc_linear_lse_noalloc(*d)
torch.cuda.synchronize()
B.mtmc_check_status()                      # reads the entry point's own status word; creates no allocating state
free1 = torch.cuda.mem_get_info()[0]
assert B.mtmc_device_alloc_count() == 0, "the library called cudaMalloc %%d times" %% B.mtmc_device_alloc_count()
assert free1 == free0, "free device memory moved by %%d bytes" %% (free0 - free1)
assert all(bool(torch.isfinite(d[3]).all()) for d in dev)
print("NOALLOC_CHILD_OK")
"""


def test_noalloc_alone_in_a_process_allocates_no_device_memory():
    """In a fresh process whose only library calls are mtmc_linear_lse_noalloc (and a status check), neither the
    library's count of cudaMalloc calls nor the device's free memory changes, up to the largest supported shapes."""
    out = subprocess.run([sys.executable, "-c", _CHILD % ROOT], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "NOALLOC_CHILD_OK" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]
