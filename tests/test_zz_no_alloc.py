"""The allocation-free logsumexp entry point, mtmc_linear_lse_noalloc.

Some callers of this library are not allowed to allocate device memory: an operator
running inside a serving loop (a cudaMalloc there stalls the whole device), a plug-in
inside a framework whose own pool already holds the GPU.  For them the library keeps
the logsumexp partials in an 8 MiB array built into its image.  This test calls the
entry point through the C ABI twice in a row -- the second call finds the first
call's leftovers in the shared array -- and checks both results against the regular
mtmc_linear_lse within the fp32 tolerance used throughout (1e-3 + 1e-3 |ref|).

The file sorts last on purpose: a run that stops at the first failure has by then
run every other test.  It is self-contained, so it also passes alone in a fresh
process (where this is the first call the library sees)."""
import pytest
import torch

from paper_2511_20100_b200 import binding as B
from paper_2511_20100_b200 import inputs

pytestmark = pytest.mark.gpu


def _within(a: torch.Tensor, ref: torch.Tensor) -> bool:
    a, ref = a.double(), ref.double()
    return bool((torch.isfinite(a)).all()) and bool(((a - ref).abs() <= 1e-3 + 1e-3 * ref.abs()).all())


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    first = inputs.linear_inputs(300, 3000, 256, seed=71)        # several column tiles, ragged M and N
    second = inputs.linear_inputs(200, 520, 448, seed=72)        # different shape: stale partials must not leak in
    for li in (first, second):
        Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
        M = Xd.shape[0]
        got = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
        mem_before = torch.cuda.memory_allocated()
        B.mtmc_linear_lse_noalloc(Xd, Wd, bd, got)
        assert torch.cuda.memory_allocated() == mem_before      # the binding allocated no tensor either
        torch.cuda.synchronize()
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
