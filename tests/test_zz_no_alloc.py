"""The allocation-free Newton-Schulz entry point, muloco_newton_schulz_static.

Some callers of this library cannot allocate device memory at the point where they
need an orthogonalisation: a framework's caching allocator may already own the whole
GPU (so a raw cudaMalloc would fail or fragment it), or the call sits in a loop that
cannot tolerate the device-wide synchronisation of cudaMalloc/cudaFree.  For them
muloco_newton_schulz_static keeps its scratch in a fixed array inside the library.

The tests call it through the C ABI several times in a row (the scratch is shared and
keeps the previous call's contents, so a later call with another layout proves that
nothing stale leaks through), with no context of the library alive, and check
  - the result against the CPU oracle's Newton-Schulz (fp32 tolerance, 1e-4),
  - that the free device memory is the same before and after the calls,
  - the result against muloco_newton_schulz in fp32 mode, twice in a row,
  - that sizes beyond the fixed scratch are refused with an explanation.
The file is collected last so that a run that stops at the first failure has already
covered every other test."""
import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import configs, synth

pytestmark = pytest.mark.gpu

NS_FP32_TOL = 1e-4      # relative Frobenius error of the fp32 Newton-Schulz, as in the other GPU tests


def _relfro(a, b):
    a = a.astype(np.float64); b = b.astype(np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


# wide, tall, ragged (cols not a multiple of 8: padded rows inside the scratch), the largest batch
# just under the 8 MiB limit, a single vector-like matrix
CASES = [(3, 128, 352), (2, 352, 128), (5, 100, 130), (64, 64, 160), (1, 8, 24)]


def test_static_entry_point_against_the_oracle_without_allocating():
    import torch
    from paper_2505_23725_b200 import binding

    rng = np.random.default_rng(2024)
    inputs = [np.stack([synth.lowrank_plus_noise(rng, m, n) for _ in range(batch)]) for batch, m, n in CASES]
    xs = [torch.from_numpy(x).cuda() for x in inputs]
    outs = [torch.empty_like(x) for x in xs]
    # Warm-up pass over every layout: the first call on a device resolves the scratch address, and
    # the first launch of each kernel variant (and of torch's fill kernel) loads its code, which may
    # take device memory once.  Everything after that must leave the free memory untouched.
    for x, o in zip(xs, outs):
        o.fill_(float("nan"))
        binding.newton_schulz_static(x, out=o)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(2):                                   # every layout twice, back to back
        for x, o in zip(xs, outs):
            o.fill_(float("nan"))
            binding.newton_schulz_static(x, out=o)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the allocation-free entry point changed the free device memory"
    for x, o in zip(inputs, outs):
        got = o.cpu().numpy()
        for b in range(x.shape[0]):
            assert _relfro(got[b], O.newton_schulz(x[b])) < NS_FP32_TOL


def test_static_entry_point_matches_regular_entry_point_twice_in_a_row():
    import torch
    from paper_2505_23725_b200 import binding

    w = configs.Workload("ns-only", K=1, H=1, J=1, tensors=[], muon_lr=0.02, muon_beta=0.95, muon_wd=0.0,
                         outer_lr=1.0, outer_momentum=0.0)
    ctx = binding.MuLoCo(w, "cuda:0", init=[])
    rng = np.random.default_rng(7)
    cases = [(3, 128, 352), (2, 352, 128)]          # wide, then tall: different scratch layouts back to back
    for batch, m, n in cases:
        X = torch.from_numpy(np.stack([synth.lowrank_plus_noise(rng, m, n) for _ in range(batch)])).cuda()
        want = ctx.newton_schulz(X, ns_mode="fp32")
        got = binding.newton_schulz_static(X)
        torch.cuda.synchronize()
        ctx.sync_status()
        for b in range(batch):
            assert _relfro(got[b].cpu().numpy(), want[b].cpu().numpy()) < NS_FP32_TOL
    ctx.close()


def test_static_entry_point_refuses_what_does_not_fit():
    import torch
    from paper_2505_23725_b200 import binding

    big = torch.zeros(1, 2048, 2048, device="cuda")
    with pytest.raises(binding.MulocoError) as e:
        binding.newton_schulz_static(big)
    assert e.value.status == binding.ESHAPE and "scratch" in str(e.value)
    with pytest.raises(binding.MulocoError) as e:      # 64 matrices that together exceed the 8 MiB
        binding.newton_schulz_static(torch.zeros(64, 64, 200, device="cuda"))
    assert e.value.status == binding.ESHAPE and "scratch" in str(e.value)
    with pytest.raises(binding.MulocoError):           # more matrices than the descriptor table holds
        binding.newton_schulz_static(torch.zeros(65, 8, 8, device="cuda"))
