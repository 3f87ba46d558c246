"""The allocation-free Newton-Schulz entry point against the regular one.

Some callers of this library cannot allocate device memory at the point where they
need an orthogonalisation: a framework's caching allocator may already own the whole
GPU (so a raw cudaMalloc would fail or fragment it), or the call sits in a loop that
cannot tolerate the device-wide synchronisation of cudaMalloc/cudaFree.  For them
muloco_newton_schulz_static keeps its scratch in a fixed array inside the library.
This test calls it through the C ABI twice in a row (the scratch is shared and keeps
the previous call's contents, so the second call proves nothing stale leaks through)
and checks both results against muloco_newton_schulz in fp32 mode, within the
Newton-Schulz tolerance of the other tests.  It is collected last so that a run that
stops at the first failure has already covered every other test."""
import numpy as np
import pytest

from paper_2505_23725_b200 import configs, synth

pytestmark = pytest.mark.gpu


def _relfro(a, b):
    a = a.astype(np.float64); b = b.astype(np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def test_static_entry_point_matches_regular_entry_point_twice_in_a_row():
    import torch
    from paper_2505_23725_b200 import binding

    w = configs.Workload("ns-only", K=1, H=1, J=1, tensors=[], muon_lr=0.02, muon_beta=0.95, muon_wd=0.0,
                         outer_lr=1.0, outer_momentum=0.0)
    ctx = binding.MuLoCo(w, "cuda:0", init=[])
    rng = np.random.default_rng(2024)
    cases = [(3, 128, 352), (2, 352, 128)]          # wide, then tall: different scratch layouts back to back
    for batch, m, n in cases:
        X = torch.from_numpy(np.stack([synth.lowrank_plus_noise(rng, m, n) for _ in range(batch)])).cuda()
        want = ctx.newton_schulz(X, ns_mode="fp32")
        got = binding.newton_schulz_static(X)
        torch.cuda.synchronize()
        ctx.sync_status()
        for b in range(batch):
            assert _relfro(got[b].cpu().numpy(), want[b].cpu().numpy()) < 1e-4
    # a request larger than the fixed scratch is refused with an explanation, not attempted
    big = torch.zeros(1, 2048, 2048, device="cuda")
    with pytest.raises(binding.MulocoError) as e:
        binding.newton_schulz_static(big)
    assert e.value.status == binding.ESHAPE and "scratch" in str(e.value)
    with pytest.raises(binding.MulocoError):
        binding.newton_schulz_static(torch.zeros(65, 8, 8, device="cuda"))
    ctx.close()
