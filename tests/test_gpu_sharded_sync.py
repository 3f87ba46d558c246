"""Worker-sharded outer synchronisation on the GPU (three library calls around a reduce-scatter and
an all-gather; Algorithm 1's all-reduce of the outer delta, Section 2 "Collectives for compressed
communication").  One GPU is available, so:
  - the NCCL path runs with a one-rank communicator and must equal muloco_outer_sync bit for bit
    and the oracle within 1e-6 (every quantiser variant, error feedback, streaming fragments);
  - the two-GPU arithmetic is emulated by two contexts on the same GPU holding half of the workers
    each, with the two collectives done by torch additions and concatenations (plain kernels, none
    waits on another), and must match the oracle over all workers.
Not tested on more than one GPU."""
import socket

import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import configs, synth
from helpers import oracle_for, gpu_for, assert_close_1e6

pytestmark = pytest.mark.gpu

SHAPES = [(128, 352), (352, 128), (5, 100), (3, 7), (1, 1000), (1, 129), (64, 128), (257, 131)]


def _np(t):
    return t.detach().float().cpu().numpy()


def _workload(K, quant, stages=1, ef=False, J=1, shapes=SHAPES):
    ts = [configs.Tensor(f"t{i}", r, c, configs.MUON if min(r, c) > 1 else configs.ADAMW, i % J)
          for i, (r, c) in enumerate(shapes)]
    return configs.Workload("sync", K=K, H=J, J=J, tensors=ts, muon_lr=0.02, muon_beta=0.9, muon_wd=0.0,
                            outer_lr=0.7, outer_momentum=0.9, quant_bits=quant, quant_stages=stages,
                            error_feedback=ef, ns_mode="fp32")


@pytest.fixture(scope="module")
def nccl_one_rank():
    import torch
    import torch.distributed as dist
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda:0"))
    yield dist
    dist.destroy_process_group()


def _drift(rng, gpus, orc, K, rnd):
    import torch
    for k in range(K):
        for i, t in enumerate(gpus[0].w.tensors):
            d = (rng.standard_normal((t.rows, t.cols)) * 10.0 ** rng.uniform(-4, -1)).astype(np.float32)
            if i == 2 and rnd == 0:
                d[1, :] = 0.0
            tk = _np(gpus[0].theta_g[i]) + d
            for g in gpus:
                g.theta_k[k][i].copy_(torch.from_numpy(tk).cuda())
            if orc is not None:
                orc.theta_k[k][i][...] = tk


@pytest.mark.parametrize("K", [1, 2, 4, 5, 16])
@pytest.mark.parametrize("quant,stages,ef", [(0, 1, False), (8, 1, False), (4, 1, False), (4, 2, False), (2, 2, False),
                                              (8, 2, True)])
def test_one_rank_nccl_path_equals_the_fused_sync_bit_for_bit(nccl_one_rank, K, quant, stages, ef):
    dist = nccl_one_rank
    w = _workload(K, quant, stages, ef, J=2)
    rng = np.random.default_rng(900 + K + quant)
    init = [rng.standard_normal((t.rows, t.cols)).astype(np.float32) * 0.02 for t in w.tensors]
    fused, shard = gpu_for(w, init), gpu_for(w, init)
    orc = oracle_for(w, init) if stages == 1 else None         # the benchmark form has a whole-sync oracle
    for rnd in range(3):
        _drift(rng, [fused, shard], orc, K, rnd)
        wire = 0
        for f in range(w.J):
            fused.outer_sync(f)
            wire += shard.sharded_outer_sync(f, dist)
        if orc is not None:
            orc.outer_sync(-1)
        fused.sync_status(); shard.sync_status()
        assert wire == 0                                       # one rank: nothing crosses a link
        for i in range(fused.n):
            assert np.array_equal(_np(shard.theta_g[i]), _np(fused.theta_g[i])), f"theta {i} round {rnd}"
            assert np.array_equal(_np(shard.outer_u[i]), _np(fused.outer_u[i])), f"u {i} round {rnd}"
            for k in range(K):
                assert np.array_equal(_np(shard.theta_k[k][i]), _np(shard.theta_g[i]))
                if ef:
                    assert np.array_equal(_np(shard.ef[k][i]), _np(fused.ef[k][i])), f"E {k} {i}"
            if orc is not None:
                assert_close_1e6(_np(shard.theta_g[i]), orc.theta_g[i], f"theta_g {i} round {rnd}")
                assert_close_1e6(_np(shard.outer_u[i]), orc.outer_u[i], f"u {i} round {rnd}")
                orc.theta_g[i][...] = _np(shard.theta_g[i]); orc.outer_u[i][...] = _np(shard.outer_u[i])
    assert fused.get_state() == shard.get_state()              # the sync counters advance alike
    fused.close(); shard.close()


@pytest.mark.parametrize("K_total,G", [(2, 2), (8, 2), (16, 4), (6, 3)])
def test_two_and_more_ranks_emulated_on_one_gpu_match_the_oracle(K_total, G):
    import torch
    Kl = K_total // G
    w_all = _workload(K_total, 0)
    w_loc = _workload(Kl, 0)
    rng = np.random.default_rng(40 + K_total)
    init = [rng.standard_normal((t.rows, t.cols)).astype(np.float32) * 0.02 for t in w_all.tensors]
    ranks = [gpu_for(w_loc, init) for _ in range(G)]
    orc = oracle_for(w_all, init)
    for rnd in range(2):
        for k in range(K_total):
            for i, t in enumerate(w_all.tensors):
                d = (rng.standard_normal((t.rows, t.cols)) * 10.0 ** rng.uniform(-4, -1)).astype(np.float32)
                orc.theta_k[k][i][...] = orc.theta_g[i] + d
                ranks[k // Kl].theta_k[k % Kl][i].copy_(torch.from_numpy(orc.theta_k[k][i]).cuda())
        stage_n, shard_n = ranks[0].shard_layout(-1, G, 0)
        assert stage_n == G * shard_n and shard_n % 128 == 0
        stages = [r.new_buffer(stage_n) for r in ranks]
        for r, st in zip(ranks, stages):
            r.shard_delta(-1, G, st)
        total = stages[0].clone()
        for st in stages[1:]:
            total += st                                        # what the reduce-scatter sums
        shards = []
        for g, r in enumerate(ranks):
            out = r.new_buffer(shard_n)
            r.shard_step(-1, G, g, total[g * shard_n:(g + 1) * shard_n].contiguous(), out)
            shards.append(out)
        theta_all = torch.cat(shards)                          # what the all-gather delivers
        for r in ranks:
            r.shard_broadcast(-1, G, theta_all)
            r.sync_status()
        orc.outer_sync(-1)
        units = 0
        for i, t in enumerate(w_all.tensors):
            ref = orc.theta_g[i]
            for r in ranks:
                assert_close_1e6(_np(r.theta_g[i]), ref, f"theta_g {i} round {rnd}")
                assert np.array_equal(_np(r.theta_g[i]), _np(ranks[0].theta_g[i]))       # all ranks agree
                for k in range(Kl):
                    assert np.array_equal(_np(r.theta_k[k][i]), _np(r.theta_g[i]))
            # u lives on the shard's owner only: element e of this tensor belongs to unit units + e // 128
            flat_u = np.concatenate([_np(r.outer_u[i]).reshape(-1)[None] for r in ranks])
            owner = (units + np.arange(t.rows * t.cols) // 128) // (shard_n // 128)
            got_u = flat_u[owner, np.arange(t.rows * t.cols)].reshape(t.rows, t.cols)
            assert_close_1e6(got_u, orc.outer_u[i], f"u {i} round {rnd}")
            units += -(-(t.rows * t.cols) // 128)
            orc.theta_g[i][...] = _np(ranks[0].theta_g[i])
            orc.outer_u[i][...] = got_u
            # the oracle's u is whole; give every rank the owner's values so the next round starts alike
            for r in ranks:
                r.outer_u[i].copy_(torch.from_numpy(got_u).cuda())
    for r in ranks:
        r.close()


def test_sharded_sync_argument_errors(nccl_one_rank):
    import dataclasses
    from paper_2505_23725_b200 import binding
    w = dataclasses.replace(_workload(2, 8, shapes=[(8, 256)]), quant_block=0)
    g = gpu_for(w, [np.zeros((8, 256), np.float32)])
    with pytest.raises(binding.MulocoError) as e:
        g.sharded_outer_sync(-1, nccl_one_rank)                # row-wise quantisation is not available sharded
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.MulocoError):
        g.shard_layout(-1, 2, 2)                               # rank outside the world
    g.close()


def test_config1_full_size_sharded_sync_equals_the_fused_sync(nccl_one_rank):
    """The benchmark's 150M-shaped workload at full size (8 replicas of 134M parameters, two
    inner steps with the benchmark's gradient recipe, then the sync): the three-pass path over a
    one-rank NCCL communicator must leave theta, u and every replica bit-equal to the fused kernel."""
    import torch
    from paper_2505_23725_b200 import binding
    w = configs.workload(1)
    outs = []
    for sharded in (False, True):
        opt = binding.MuLoCo(w, "cuda:0", init_seed=11, alloc_grads=True)
        for step in range(2):
            synth.torch_fill_gradients(opt.grads, w.tensors, w.K, 100 + step, opt.device)
            opt.inner_step(-1, None, 1.0)
        if sharded:
            assert opt.sharded_outer_sync(-1, nccl_one_rank) == 0      # one rank: nothing on the wire
        else:
            opt.outer_sync(-1)
        opt.sync_status()
        # per tensor (the flat buffers have uninitialised padding between tensors)
        outs.append([(opt.theta_g[i].clone(), opt.outer_u[i].clone(), opt.theta_k[0][i].clone(),
                      opt.theta_k[w.K - 1][i].clone()) for i in range(opt.n)])
        opt.close()
        del opt
        torch.cuda.empty_cache()
    for i, (fused, shard) in enumerate(zip(outs[0], outs[1])):
        for a, b, what in zip(fused, shard, ("theta", "u", "replica 0", "replica K-1")):
            assert torch.equal(a, b), f"tensor {i}: {what}"
        assert torch.equal(shard[2], shard[0]) and torch.equal(shard[3], shard[0])
