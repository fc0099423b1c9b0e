"""The allocation-free exchange entry point against the ordinary compress + decompress pair.

Some users of the library call it from places where device memory cannot be allocated (inside a
latency-critical loop, or when another framework's caching allocator already owns the GPU's
memory).  For them varco_exchange_noalloc keeps its packed rows in a fixed array inside the
library.  This test calls it through the C ABI twice in a row -- the array is shared between calls
and keeps the previous call's contents -- and expects bit-identical halo rows each time.
Collected last on purpose, so that a failure here cannot hide any other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2406_17611_b200 import binding as vb
from paper_2406_17611_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_exchange_matches_compress_decompress_twice(orc):
    wl = synth.make_workload("c3", 0.004)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload()
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    perm = plan.perm()
    # the last two calls keep whole rows (k = F): 100 bf16 and 64 fp32 values per copy, both inside the scratch
    calls = [(100, (4, 1), (7, 1, 0), torch.bfloat16), (256, (16, 1), (7, 2, 1), torch.bfloat16),
             (64, (385, 4), (7, 3, 0), torch.float32), (100, (1, 1), (7, 4, 1), torch.bfloat16),
             (64, (1, 1), (7, 5, 0), torch.float32)]
    assert plan.H_total * 104 * 2 <= vb.NOALLOC_SCRATCH_BYTES and plan.H_total * 64 * 4 <= vb.NOALLOC_SCRATCH_BYTES
    for rep in range(2):
        for F, ratio, key, dt in calls:
            vec = 4 if dt == torch.float32 else 8
            ld = (F + vec - 1) // vec * vec
            X = synth.normal_features(wl.n, F, 11 + rep, dt == torch.bfloat16)
            Xd = torch.zeros((wl.n, ld), dtype=dt)
            Xd[:, :F] = torch.from_numpy(X[perm]).to(dt)
            Xd = Xd.cuda()
            packed, want_bytes = vb.varco_compress(plan, Xd, F, ratio, key)
            want = vb.varco_decompress(plan, packed, F, ratio, key, ld=ld)
            out = torch.full((plan.H_total, ld), 7.0, dtype=dt, device="cuda")   # caller-owned output
            before = torch.cuda.memory_allocated()
            got_bytes = vb.varco_exchange_noalloc(plan, Xd, F, ratio, key, out)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert got_bytes == want_bytes
            assert torch.equal(out[:, :F], want[:, :F])
            # and against the oracle itself: decompress(compress(X)), bit for bit, same byte count
            ref_packed, sent = g.compress(X, ratio, key)
            assert got_bytes == sent * (4 if dt == torch.float32 else 2)
            ref = g.decompress(ref_packed, F, ratio, key)
            assert np.array_equal(out[:, :F].to(torch.float64).cpu().numpy(), ref)


def test_noalloc_exchange_rejects_sizes_beyond_its_scratch():
    wl = synth.make_workload("c2r", 0.2)     # ~130k halo copies: at 256 fp32 values each they need > 32 MiB
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload()
    F = 256
    assert plan.H_total * F * 4 > vb.NOALLOC_SCRATCH_BYTES
    X = torch.zeros((wl.n, F), dtype=torch.float32, device="cuda")
    out = torch.zeros((plan.H_total, F), dtype=torch.float32, device="cuda")
    with pytest.raises(vb.VarcoError) as e:
        vb.varco_exchange_noalloc(plan, X, F, (1, 1), (0, 0, 0), out)
    assert e.value.status == -6
    # a ratio that brings the packed rows under the limit is accepted
    assert vb.varco_exchange_noalloc(plan, X, F, (64, 1), (0, 0, 0), out) == plan.H_total * 4 * 4
    torch.cuda.synchronize()
