"""The benchmark's multi-rank plumbing on CPU: two gloo ranks, no GPU.

Batch rows are independent, so ranks share nothing on the data path; what the ranks do
exchange is the timing (maximum over ranks) and, in a sharded deployment, the per-row
controller signals.  Both are exercised here with world_size 2.
"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    from paper_2510_02358_b200 import binding as dsp
    from paper_2510_02358_b200 import workloads as wl
    # timing: the job's time is the slowest rank's
    ms = bench.reduce_max_ms(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    # each rank owns different batch rows of the same workload
    w = wl.CONFIGS[3].scaled(B=2, L=3, V=512)
    mine = wl.make_inputs(w, step=bench.rank_seed_base(rank))
    lat = oracle.lattice_build(mine["draft"], w.K)
    cps = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, mine["prev_token"],
                            mine["table"], W=w.W, lam=w.lam, table_log2=mine["table_log2"],
                            hash_seed=mine["hash_seed"], V=w.V)
    ver = oracle.verify(mine["target"], mine["draft"], cps.path, cps.path_len, mine["mode"], mine["u"])
    # the controller needs the batch means over ALL rows: gather the two [B] int arrays
    sig = torch.stack([ver.accepted_len, lat.gen_len]).int()
    allsig = [torch.empty_like(sig) for _ in range(world)]
    dist.all_gather(allsig, sig)
    acc = torch.cat([s[0] for s in allsig])
    gen = torch.cat([s[1] for s in allsig])
    st, prm = dsp.dsp_adl_init(8, 32, 8.0, 0.5, 8)
    k = dsp.dsp_adl_update(st, prm, acc, gen)
    ks = [torch.zeros(1, dtype=torch.int32) for _ in range(world)]
    dist.all_gather(ks, torch.tensor([k], dtype=torch.int32))
    out[rank] = dict(ms=ms, k=[int(x) for x in ks], draft_sum=float(mine["draft"].float().sum()),
                     value=bench.whole_job_steps_per_s(world, 20, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    world = 2
    port = 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    r0, r1 = out[0], out[1]
    assert r0["ms"] == r1["ms"] == 15.0                       # max over ranks
    assert r0["value"] == r1["value"] == 2 * 20 / 0.015       # both ranks' steps over the slowest time
    assert r0["k"] == r1["k"] and r0["k"][0] == r0["k"][1]    # every rank derives the same next length
    assert r0["draft_sum"] != r1["draft_sum"]                 # different rows per rank


def _gather_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from types import SimpleNamespace
    from paper_2510_02358_b200 import binding as dsp
    B, L, K = 2, 3, 4
    # stand-ins for one rank's slice records (their content is the kernels' business, the layout is the host's)
    rec = SimpleNamespace(sums=torch.full((B, L, dsp.SHARD_SUMS_BYTES), rank + 1, dtype=torch.uint8),
                          keys=torch.arange(B * L * K, dtype=torch.int64).view(B, L, K) + 1000 * rank,
                          status=torch.full((B,), 32 * rank, dtype=torch.int32))
    g = dsp.gather_shard_records(rec)
    out[rank] = dict(sums=g.sums.clone(), keys=g.keys.clone(), status=g.status.clone())
    dist.barrier()
    dist.destroy_process_group()


def test_slice_records_are_gathered_slice_major_on_every_rank():
    """The vocabulary-sharded lattice: rank r holds slice r; every rank ends with the [G, ...] buffers
    that dsp_lattice_merge reads, slice r at index r."""
    world = 2
    port = 31500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_gather_worker, args=(world, port, out), nprocs=world, join=True)
    for r in range(world):
        o = out[r]
        assert tuple(o["sums"].shape) == (world, 2, 3, 24) and tuple(o["keys"].shape) == (world, 2, 3, 4)
        assert tuple(o["status"].shape) == (world, 2)
        for s in range(world):
            assert (o["sums"][s] == s + 1).all() and o["keys"][s, 0, 0, 0] == 1000 * s
            assert (o["status"][s] == 32 * s).all()
    assert torch.equal(out[0]["keys"], out[1]["keys"])


class _WallTimer:
    device = torch.device("cpu")

    def __init__(self):
        self.t = None

    def record(self):
        import time
        self.t = time.perf_counter()

    def sync(self):
        pass

    def elapsed_ms(self, other):
        return (other.t - self.t) * 1e3


def _exchange_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from types import SimpleNamespace
    import bench
    from paper_2510_02358_b200 import binding as dsp
    B, L, K, V = 2, 3, 4, 1000
    lo, hi = bench.vocab_slice(V, world, rank)
    seen = {}

    def shard():                      # stand-in for dsp_lattice_shard: the records name their slice
        return SimpleNamespace(sums=torch.full((B, L, dsp.SHARD_SUMS_BYTES), rank + 1, dtype=torch.uint8),
                               keys=torch.full((B, L, K), lo, dtype=torch.int64),
                               status=torch.zeros((B,), dtype=torch.int32))

    def merge(a):                     # stand-in for dsp_lattice_merge: every slice must be there, in order
        seen["los"] = a.keys[:, 0, 0, 0].tolist()
        seen["shape"] = tuple(a.sums.shape)

    res = bench.sharded_exchange_leg(shard, dsp.gather_shard_records, merge, _WallTimer, 3, dist)
    out[rank] = dict(res=res, los=seen["los"], shape=seen["shape"], slice=(lo, hi))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_exchange_leg_of_the_benchmark_on_two_ranks():
    """The bench leg for several GPUs (slice -> all-gather of the records -> merge) with stand-in kernels:
    the slices tile the vocabulary, every rank merges all slices' records in slice order, and the
    reported times are the same on every rank (maximum over ranks)."""
    world = 2
    port = 33500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_exchange_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0]["slice"][0] == 0 and out[0]["slice"][1] == out[1]["slice"][0] and out[1]["slice"][1] == 1000
    assert out[0]["slice"][1] % 8 == 0
    for r in range(world):
        assert out[r]["los"] == [out[0]["slice"][0], out[1]["slice"][0]] and out[r]["shape"][0] == world
        assert set(out[r]["res"]) == {"shard_ms", "gather_ms", "merge_ms"}
    assert out[0]["res"] == out[1]["res"]
