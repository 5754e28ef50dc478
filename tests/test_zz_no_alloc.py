"""The allocation-free step-size entry point (`nsd_step_size_noalloc`).

Hosts that may not allocate device memory when they call the library -- a server whose
memory was handed out at start-up, a real-time loop that cannot afford cudaMalloc's implicit
synchronisation -- get Delta = s * std(delta) from a call that owns no context and uses a
fixed scratch array inside the library. This file checks that call against the regular
`nsd_quantize` entry point and against the CPU oracle's step size, twice in a row (the scratch array keeps the previous call's
contents, so the second call is the one that would show stale state), for both storage types,
and that a tensor beyond the stated limit is refused before anything runs.

It is named so that pytest collects it after every other test file."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


def _reference_step(ctx, d, scale):
    import paper_2004_04729_b200 as dbp
    q = dbp.nsd_quantize(ctx, d, 0, scale)
    torch.cuda.synchronize()
    return float(q.delta.item())


def test_noalloc_step_matches_regular_entry_point_twice():
    import paper_2004_04729_b200 as dbp
    ctx = dbp.Context(0)
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    cases = [
        (torch.from_numpy(wl.config3(batch=4).delta).cuda(), 2.0),                        # 1 Mi fp32
        (torch.from_numpy(wl.config1().delta).cuda().to(torch.bfloat16), 5.0),            # small, bf16
        (torch.from_numpy(wl.laplace(3, 1, 70001, 1e-3).astype(np.float32)).cuda(), 2.0), # ragged tail
    ]
    for d, scale in cases:
        want = _reference_step(ctx, d, scale)
        # the oracle sees the values the kernel sees (bf16 widens exactly to fp32)
        exact = float(oracle.step_size(d.float().cpu().numpy(), scale))
        for _ in range(2):                       # two calls in a row on the shared scratch
            out.fill_(-1.0)
            dbp.nsd_step_size_noalloc(d, scale, out)
            torch.cuda.synchronize()
            got = float(out.item())
            assert want > 0 and abs(got - want) <= 1e-6 * want, (got, want)
            assert abs(got - exact) <= 1e-6 * exact, (got, exact)
    # sigma = 0 is not an error: all-zero input, and a constant that is no binary fraction
    for value in (0.0, 0.1):
        dbp.nsd_step_size_noalloc(torch.full((4099,), value, device="cuda"), 2.0, out)
        torch.cuda.synchronize()
        assert out.item() == 0.0
    ctx.close()


def test_noalloc_refuses_sizes_beyond_its_limit_and_bad_arguments():
    import paper_2004_04729_b200 as dbp
    d = torch.ones(64, device="cuda")
    out = torch.full((1,), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(dbp.DbpError) as e:       # the size check comes before any launch
        dbp.nsd_step_size_noalloc(d, 2.0, out, numel=(1 << 31) + 1)
    assert e.value.status == -7
    with pytest.raises(dbp.DbpError) as e:
        dbp.nsd_step_size_noalloc(d, 0.0, out)
    assert e.value.status == -1
    torch.cuda.synchronize()
    assert out.item() == 7.0                     # nothing was enqueued
