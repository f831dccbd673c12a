"""The multi-rank plumbing on CPU: two ``gloo`` processes shard the samples, each runs its own
(oracle) cache on its shard with no exchange on the data path, and only the timing reduction and the
optional decision gather cross ranks. Checks that the sharded decisions equal the unsharded ones."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _inputs(B, n, seed=11):
    g = torch.Generator().manual_seed(seed)
    feats = [torch.randn(B, n, generator=g).numpy().copy() for _ in range(3)]
    noise = torch.tensor([0.0, 0.01, 0.3, 1.0, 0.02])[:B].view(B, 1)
    fresh_noise = (torch.randn(B, n, generator=g) * noise).numpy()
    return feats, fresh_noise


def _decisions(sample_ids, feats, fresh_noise, n):
    from oracle import speca_oracle as O
    B = len(sample_ids)
    if B == 0:
        return [], []
    cache = O.OracleCache([n], B, 2, O.F32)
    for k, t in enumerate([1.0, 0.9, 0.8]):
        cache.update([feats[k][sample_ids]], [t] * B)
        cache.commit_step()
    pred = cache.forecast_entry(0, [0.75] * B)
    fresh = (pred + fresh_noise[sample_ids]).astype(np.float32)
    err, acc, _ = cache.verify(fresh, [0.75] * B, [0.05] * B)
    return [float(e) for e in err], [int(a) for a in acc]


def _worker(rank, world, port, out_dir):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2509_11628_b200 import dist as D
    info = D.init("gloo")
    assert (info.rank, info.world) == (rank, world) and info.is_main == (rank == 0)
    B, n = 5, 257
    feats, fresh_noise = _inputs(B, n)
    mine = D.shard_samples(B, world, rank)
    D.barrier()
    err, acc = _decisions(mine, feats, fresh_noise, n)
    D.barrier()
    slowest = D.max_over_ranks(10.0 + rank)
    total = D.sum_over_ranks(len(mine))
    everyone = D.gather_decisions(acc)
    assert slowest == 10.0 + (world - 1)
    assert total == B
    flat = [a for part in everyone for a in part]
    if rank == 0:
        torch.save({"acc": flat, "err_rank0": err, "shard0": mine}, os.path.join(out_dir, "r0.pt"))
    D.shutdown()


def test_two_ranks_shard_samples_without_a_data_path_collective(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = torch.load(os.path.join(str(tmp_path), "r0.pt"))
    B, n = 5, 257
    feats, fresh_noise = _inputs(B, n)
    err_all, acc_all = _decisions(list(range(B)), feats, fresh_noise, n)
    assert got["acc"] == acc_all            # per-sample decisions do not depend on the sharding
    assert got["shard0"] == [0, 1, 2]
    # a sample's error depends on that sample alone; the oracle adds up in a thread-count-dependent
    # order, so two processes may differ in the last place of a double
    assert got["err_rank0"] == pytest.approx(err_all[:3], rel=1e-12, abs=0.0)
    assert acc_all[0] == 1 and acc_all[3] == 0


def test_shard_samples_is_a_balanced_partition():
    from paper_2509_11628_b200 import dist as D
    for n in (1, 5, 8, 16, 64):
        for world in (1, 2, 3, 4, 8):
            parts = [D.shard_samples(n, world, r) for r in range(world)]
            flat = [i for p in parts for i in p]
            assert flat == list(range(n))
            sizes = [len(p) for p in parts]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_reductions_are_identities():
    from paper_2509_11628_b200 import dist as D
    assert not dist.is_initialized()
    assert D.max_over_ranks(3.5) == 3.5 and D.sum_over_ranks(2.0) == 2.0
    assert D.gather_decisions([1, 0]) == [[1, 0]]
    D.barrier()


# ---------------------------------------------------------------------------------------------
# token-sharded verification: two ranks each hold half the tokens of the verification entry; the
# only exchange is the combination of 4 doubles per sample
# ---------------------------------------------------------------------------------------------

def _verify_inputs(B, tokens, dim, seed=5):
    g = torch.Generator().manual_seed(seed)
    feats = [torch.randn(B, tokens, dim, generator=g).numpy().copy() for _ in range(3)]
    fresh_noise = (torch.randn(B, tokens, dim, generator=g) * torch.tensor([0.0, 0.02, 0.5]).view(B, 1, 1)).numpy()
    return feats, fresh_noise


def _shard_sums(metric, feats, fresh_noise, tok0, ntok, nan_at=None):
    """Oracle: tables over tokens [tok0, tok0+ntok) only, forecast, running values of the metric."""
    from oracle import speca_oracle as O
    B, _, dim = feats[0].shape
    n = ntok * dim
    cache = O.OracleCache([n], B, 2, O.F32)
    sl = slice(tok0, tok0 + ntok)
    for k, t in enumerate([1.0, 0.9, 0.8]):
        cache.update([np.ascontiguousarray(feats[k][:, sl]).reshape(B, n)], [t] * B)
        cache.commit_step()
    pred = cache.forecast_entry(0, [0.75] * B)
    fresh = (pred + np.ascontiguousarray(fresh_noise[:, sl]).reshape(B, n)).astype(np.float32)
    if nan_at is not None and tok0 <= nan_at < tok0 + ntok:
        fresh[1, (nan_at - tok0) * dim] = np.nan
    return np.array([O.metric_sums(metric, O.F32, pred[b], fresh[b]) + [0.0] for b in range(B)], dtype=np.float64)


def _token_worker(rank, world, port, out_dir):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2509_11628_b200 import dist as D
    D.init("gloo")
    B, tokens, dim = 3, 37, 16
    feats, fresh_noise = _verify_inputs(B, tokens, dim)
    tok0, ntok = D.shard_tokens(tokens, world, rank)
    out = {}
    for metric in (0, 1, 2, 3):
        for nan_at in (None, 30):
            sums = torch.from_numpy(_shard_sums(metric, feats, fresh_noise, tok0, ntok, nan_at))
            D.combine_verify_sums(sums, linf=(metric == 2))
            out[(metric, nan_at)] = sums.numpy().copy()
    if rank == 0:
        torch.save(out, os.path.join(out_dir, "tok.pt"))
    D.shutdown()


def test_two_ranks_token_sharded_verification_matches_unsharded(tmp_path):
    from oracle import speca_oracle as O
    from paper_2509_11628_b200 import dist as D
    port = _free_port()
    mp.spawn(_token_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = torch.load(os.path.join(str(tmp_path), "tok.pt"), weights_only=False)
    B, tokens, dim = 3, 37, 16
    feats, fresh_noise = _verify_inputs(B, tokens, dim)
    assert [D.shard_tokens(tokens, 2, r) for r in range(2)] == [(0, 19), (19, 18)]
    for metric in (0, 1, 2, 3):
        for nan_at in (None, 30):
            whole = _shard_sums(metric, feats, fresh_noise, 0, tokens, nan_at)
            for b in range(B):
                e_want = O.metric_from_sums(metric, whole[b][:3])
                e_got = O.metric_from_sums(metric, got[(metric, nan_at)][b][:3])
                if nan_at is not None and b == 1:
                    assert np.isnan(e_want) and np.isnan(e_got) and not O.accept(e_got, 1e30)
                else:
                    assert e_got == pytest.approx(e_want, rel=1e-12, abs=1e-15)
                    assert O.accept(e_got, 0.05) == O.accept(e_want, 0.05)
