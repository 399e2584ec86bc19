"""pact_prune_static, the percentile split for callers that cannot allocate device memory.

Some hosts of the library have no way to obtain a workspace: they run inside another framework's
callback, or are handed tensors but no allocator, or live in a process whose device memory is
already fully parcelled out.  For them the scratch of the split is a fixed array inside the
library.  This test calls that entry point through the C ABI twice in a row (the second call finds
the array as the first one left it, with a different N and pruning fraction) and requires bit-equal
outputs to pact_prune, which uses a caller workspace, and to the CPU oracle's split.  Larger inputs go
through the other variants of the kernel (keys in registers, in shared memory, re-read), and one case
runs in a process of its own in which nothing else has touched the library, so that the entry point's
own first-call set-up is what makes the large launch possible.  The file sorts last so that a failure
here cannot hide the result of any other test in a run that stops at the first failure.
"""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import pact_oracle as orc

pytestmark = pytest.mark.gpu


def _run_both(pb, ctx, score, lam):
    N = score.numel()
    p = pb.make_params(lam=lam)

    def outputs():
        return (torch.full((N,), 7, dtype=torch.uint8, device="cuda"),
                torch.full((N,), -5, dtype=torch.int32, device="cuda"),
                torch.full((N,), -5, dtype=torch.int32, device="cuda"),
                torch.full((2,), -5, dtype=torch.int32, device="cuda"))

    ref = outputs()
    ctx.pact_prune(score, p, *ref)
    got = outputs()
    pb.pact_prune_static(score, p, *got)
    torch.cuda.synchronize()
    q, m = ref[3].cpu().tolist()
    assert got[3].cpu().tolist() == [q, m] and q + m == N
    assert torch.equal(got[0], ref[0])
    assert torch.equal(got[1][:q], ref[1][:q]) and torch.equal(got[2][:m], ref[2][:m])
    # and against the oracle's split of the same float32 scores (Eq. 3-4)
    _, keep, kept, pruned = orc.split(score.cpu().numpy(), lam)
    assert np.array_equal(got[0].cpu().numpy().astype(bool), keep)
    assert np.array_equal(got[1][:q].cpu().numpy(), kept) and np.array_equal(got[2][:m].cpu().numpy(), pruned)
    return q, m


def test_static_scratch_split_matches_workspace_split_twice_in_a_row():
    from paper_2504_08966_b200 import binding as pb
    ctx = pb.Context(256, 2, 2, 32, torch.bfloat16, torch.bfloat16)
    g = torch.Generator().manual_seed(5)
    a = torch.rand(5000, generator=g).cuda()
    a[17] = a[4000] = a[99]                        # ties
    a[3] = -0.25
    b = torch.rand(1237, generator=g).cuda()
    q1, m1 = _run_both(pb, ctx, a, 0.5)
    q2, m2 = _run_both(pb, ctx, b, 0.3)            # second call: smaller N, stale scratch from the first
    assert m1 == 2500 and m2 == 371
    q3, _ = _run_both(pb, ctx, a, 0.0)             # nothing pruned
    assert q3 == 5000


@pytest.mark.parametrize("N", [12000, 40000, 65536])
def test_static_scratch_split_at_the_sizes_of_the_other_kernel_variants(N):
    """Up to 8192 scores a thread keeps 8 keys in registers, up to 16384 it keeps 16, beyond that the keys
    live in shared memory; 65536 is the largest input the array admits."""
    from paper_2504_08966_b200 import binding as pb
    ctx = pb.Context(256, 2, 2, 32, torch.bfloat16, torch.bfloat16)
    g = torch.Generator().manual_seed(N)
    a = (torch.rand(N, generator=g) * torch.rand(N, generator=g)).cuda()
    a[N // 3] = a[N // 2]                          # a tie
    q, m = _run_both(pb, ctx, a, 0.37)
    assert m <= int(0.37 * N + 1e-6)
    _run_both(pb, ctx, a[: N // 2].contiguous(), 0.8)   # second call in a row, stale scratch from the first


_FRESH = r"""
import sys
import numpy as np, torch
sys.path.insert(0, sys.argv[1])
from paper_2504_08966_b200 import binding as pb
from oracle import pact_oracle as orc
N, lam = 40000, 0.61
g = torch.Generator().manual_seed(7)
score = torch.rand(N, generator=g).cuda()
keep = torch.full((N,), 7, dtype=torch.uint8, device="cuda")
kept = torch.full((N,), -5, dtype=torch.int32, device="cuda")
pruned = torch.full((N,), -5, dtype=torch.int32, device="cuda")
counts = torch.full((2,), -5, dtype=torch.int32, device="cuda")
for _ in range(2):                                 # no pact_create anywhere in this process
    pb.pact_prune_static(score, pb.make_params(lam=lam), keep, kept, pruned, counts)
    torch.cuda.synchronize()
    q, m = counts.cpu().tolist()
    _, k_o, kept_o, pruned_o = orc.split(score.cpu().numpy(), lam)
    assert q == kept_o.size and m == pruned_o.size
    assert np.array_equal(keep.cpu().numpy().astype(bool), k_o)
    assert np.array_equal(kept[:q].cpu().numpy(), kept_o) and np.array_equal(pruned[:m].cpu().numpy(), pruned_o)
print("fresh ok")
"""


def test_static_scratch_split_as_the_first_call_of_a_fresh_process():
    """No context is ever created in the child: the entry point's own first call on the device must look up
    the array's address and enable the large shared-memory launch that 40000 scores need."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _FRESH, root], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "fresh ok" in r.stdout, r.stdout + r.stderr


def test_static_scratch_split_rejects_sizes_beyond_its_array():
    import ctypes as C
    from paper_2504_08966_b200 import binding as pb
    L = pb.lib()
    n = pb.PRUNE_STATIC_MAX_N + 1
    buf = torch.zeros(n, dtype=torch.float32, device="cuda")
    i32 = torch.zeros(n, dtype=torch.int32, device="cuda")
    p = pb.make_params(lam=0.5)
    vp = lambda t: C.c_void_p(t.data_ptr())
    st = L.pact_prune_static(vp(buf), n, C.byref(p), vp(i32), vp(i32), vp(i32), vp(i32), None)
    assert st == -2
    assert L.pact_prune_static(None, 16, C.byref(p), vp(i32), vp(i32), vp(i32), vp(i32), None) == -1
    bad = pb.make_params(lam=1.5)
    assert L.pact_prune_static(vp(buf), 16, C.byref(bad), vp(i32), vp(i32), vp(i32), vp(i32), None) == -1
    torch.cuda.synchronize()
