"""fp4_root_ns_static: the Root step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits (inside another framework's
callback, in a latency-critical loop, or with a memory pool that is already spoken for), so
they cannot hand the library a workspace.  fp4_root_ns_static keeps the workspace in a static
16 MiB device array inside the library instead.  This file checks, through the C ABI, that
it gives exactly what fp4_root_ns gives with a caller-allocated workspace -- twice in a row,
because every call reuses the same array and must clear what has to start from zero -- and
that shapes beyond the array's size are refused.  It is collected last on purpose, and it
passes both on its own in a fresh process and after the rest of the suite."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_04422_b200 as fp4
from paper_2607_04422_b200 import workloads
from paper_2607_04422_b200.binding import FP4_STATIC_SCRATCH_BYTES

pytestmark = pytest.mark.gpu


def _with_workspace(G_np, steps):
    G = torch.from_numpy(G_np).cuda()
    out = torch.empty_like(G)
    ws = torch.empty(fp4.fp4_root_ns_workspace_bytes(*G_np.shape, steps), dtype=torch.uint8, device="cuda")
    fp4.fp4_root_ns(G, out, steps, None, ws)
    assert fp4.fp4_last_device_status(ws) == 0
    return out.cpu().numpy()


def test_static_scratch_matches_workspace_call_twice_in_a_row():
    # two different problems back to back: the second call sees the first call's leftovers
    cases = [(workloads.gradient_like(512, 1024, seed=21), 5),
             (workloads.lowrank_outliers(768, 384, seed=22), 3)]
    want = [_with_workspace(g, k) for g, k in cases]
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for round_ in range(2):
        for (g, k), w in zip(cases, want):
            G = torch.from_numpy(g).cuda()
            out = torch.full_like(G, float("nan"))
            fp4.fp4_root_ns_static(G, out, k, None, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            # same kernels, same order, deterministic: the tolerance of the other parity tests
            # (2e-3 relative Frobenius) is met with equality
            got = out.cpu().numpy()
            rel = np.linalg.norm(got.astype(np.float64) - w) / np.linalg.norm(w.astype(np.float64))
            assert rel <= 2e-3 and np.array_equal(got, w), (round_, g.shape, rel)
    # and against the CPU oracle, like every other parity test of the step
    g, k = cases[1]
    ref = oracle.root_ns(g, steps=k).astype(np.float64)
    assert np.linalg.norm(got.astype(np.float64) - ref) / np.linalg.norm(ref) <= 2e-3


def test_static_scratch_refuses_what_does_not_fit():
    assert fp4.fp4_root_ns_workspace_bytes(1024, 2048, 5) <= FP4_STATIC_SCRATCH_BYTES
    assert fp4.fp4_root_ns_workspace_bytes(2048, 2048, 5) > FP4_STATIC_SCRATCH_BYTES
    G = torch.zeros((2048, 2048), device="cuda")
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_root_ns_static(G, G, 5)
    assert e.value.code == 9
    with pytest.raises(fp4.Fp4Error) as e:
        fp4.fp4_root_ns_static(torch.zeros((100, 256), device="cuda"), G, 5)
    assert e.value.code == 2
