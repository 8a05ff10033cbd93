"""lqsgd_orthonormalize_noalloc: the entry point for callers that cannot allocate device memory
(their GPU memory is fully owned by another allocator, or cudaMalloc is forbidden where they run
because it stalls the device).  It keeps its intermediate storage in a fixed array inside the
library instead of a caller workspace.  Checked here, through the C ABI, against the orthonormal
factor the regular workspace-based step produces from the same input - on two calls in a row,
because all calls share that one array and the second must not see leftovers of the first.

Collected last on purpose (file name): a failure here cannot hide another test's result."""
import numpy as np
import pytest
import torch

from oracle import lqsgd_oracle as orc
from paper_2506_17974_b200 import binding as B
from paper_2506_17974_b200 import workloads as wl
import parity as par

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _step_and_fetch(shape, rank, workers, seed):
    w = wl.Workload("noalloc", (shape,), rank=rank, bits=4, workers=workers, steps=1,
                    dist="normal", scale="fan_in", seed=seed)
    comp = B.LQSGD(w.layers, w.rank, w.bits, workers=w.workers, seed=seed)
    g = wl.draw_gradients(w, 0, device=DEV)
    comp.step(g, [torch.empty(shape, device=DEV)])
    torch.cuda.synchronize()
    raw = [comp.get_state(B.STATE_P_RAW, 0, k) for k in range(workers)]
    ref = [comp.get_state(B.STATE_P, 0, k) for k in range(workers)]
    return raw, ref


def test_no_alloc_orthonormalize_matches_workspace_path_twice():
    raw_a, ref_a = _step_and_fetch((1000, 300), 5, 2, seed=1)
    raw_b, ref_b = _step_and_fetch((333, 64), 16, 1, seed=2)      # other size and rank in between
    status = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    calls = [(raw_a[0], ref_a[0]), (raw_b[0], ref_b[0]), (raw_a[1], ref_a[1]), (raw_a[0], ref_a[0])]
    for raw, ref in calls:                                        # back-to-back calls, same stream
        out = torch.full_like(raw, float("nan"))
        B.orthonormalize_noalloc(raw, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert par.rel_fro(par.host(out), par.host(ref)) <= par.TOL
        assert par.rel_fro(par.host(out), orc.orthonormalize(par.host(raw))[0]) <= par.TOL   # and the CPU oracle's
        gram = par.host(out).astype(np.float64)
        assert np.max(np.abs(gram.T @ gram - np.eye(raw.shape[1]))) < 1e-5
    # in place
    buf = raw_a[0].clone()
    B.orthonormalize_noalloc(buf, buf)
    torch.cuda.synchronize()
    assert par.rel_fro(par.host(buf), par.host(ref_a[0])) <= par.TOL


def test_no_alloc_reports_dependent_column_and_clears_it_on_the_next_call():
    x = torch.randn(500, 3, device=DEV, generator=torch.Generator(DEV).manual_seed(4))
    x[:, 2] = x[:, 0]
    out = torch.empty_like(x)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.orthonormalize_noalloc(x, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) & B.STATUS_DEPENDENT_COLUMN
    assert float(out[:, 2].abs().max()) == 0.0
    y = torch.randn(500, 3, device=DEV, generator=torch.Generator(DEV).manual_seed(5))
    B.orthonormalize_noalloc(y, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0


@pytest.mark.parametrize("rows", [B.NOALLOC_MAX_ROWS, B.NOALLOC_MAX_ROWS - 127])
def test_no_alloc_largest_accepted_sizes(rows):
    """The last block's Gram matrix sits right before R^-1 in the fixed array: at the largest sizes the
    result must still be orthonormal, equal to the oracle's, and report no condition."""
    x = torch.randn(rows, 16, device=DEV, generator=torch.Generator(DEV).manual_seed(rows))
    out = torch.empty_like(x)
    status = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    for _ in range(2):
        B.orthonormalize_noalloc(x, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    q = par.host(out).astype(np.float64)
    assert np.max(np.abs(q.T @ q - np.eye(16))) < 1e-5
    assert par.rel_fro(q, orc.orthonormalize(par.host(x))[0]) <= par.TOL


def test_no_alloc_rejects_sizes_beyond_its_fixed_scratch():
    x = torch.zeros(8, 4, device=DEV)
    for rows, rank, code in [(B.NOALLOC_MAX_ROWS + 1, 4, B.ERR_TOO_LARGE), (8, 17, B.ERR_TOO_LARGE),
                             (0, 4, B.ERR_INVALID_ARG), (8, 0, B.ERR_INVALID_ARG)]:
        with pytest.raises(B.LqsgdError) as e:
            B.orthonormalize_noalloc(x, x, rows=rows, rank=rank)
        assert e.value.code == code
    assert "scratch" in B.load_library().lqsgd_strerror(B.ERR_TOO_LARGE).decode()
