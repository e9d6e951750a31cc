"""Data-parallel AdamA (Section 3.3, Eqs. 4-7) without a GPU.

The CUDA kernels cannot run here, so the ranks (real processes, gloo backend, world size 2)
carry fp32 CPU states and apply the library's own host-derived constants with numpy in place
of the kernels; what is under test is the multi-process protocol: the collective helper, the
R*beta2 pre-scaling, the 1/R and 1/R^2 folded into the constants, and that every rank ends
with the single-device result for N*R micro-batches (fp64 oracle)."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import paper_2305_19982_b200 as adama
from oracle import AdamAOracle
from paper_2305_19982_b200 import ddp
from parity import rel_l2

ROOT = Path(__file__).resolve().parent.parent
B1, B2, EPS, LR = 0.9, 0.999, 1e-8, 1e-3


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_allreduced_constants_fold_the_world_size():
    R, N, t = 4, 3, 7
    c1 = adama.host_constants(B1, B2, EPS, N, t, LR)
    cR = adama.host_constants(B1, B2, EPS, N, t, LR, world_size=R)
    f32 = lambda x: float(np.float32(x))
    assert cR[0] == c1[0] and cR[1] == c1[1]            # folds are rank-local: unchanged
    assert cR[2] == f32(LR / (1 - B1 ** t) / R)
    assert cR[3] == f32(1 / (1 - B2 ** t) / R ** 2)
    assert abs((cR[5] + cR[6]) - B1 / R) < 1e-14
    assert abs((cR[7] + cR[8]) - B2 / R) < 1e-14
    with pytest.raises(adama.AdamAError):
        adama.host_constants(B1, B2, EPS, N, t, LR, world_size=0)


def _rank_main(rank, world, port, n, N, steps, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(123)
    w = rng.normal(0, 0.02, n).astype(np.float32)        # same on every rank
    grads = rng.normal(0, 1e-2, (steps, world, N, n)).astype(np.float32)
    m = torch.zeros(n)
    v = torch.zeros(n)
    f = np.float32
    for step in range(steps):
        t = step + 1
        c = [f(x) for x in adama.host_constants(B1, B2, EPS, N, t, LR, world_size=world)]
        for i in range(N):                               # rank-local folds (what adama_fold does)
            g = grads[step, rank, i]
            m += torch.from_numpy(c[0] * g)
            v += torch.from_numpy((c[1] * g) * g)
        assert ddp.allreduce_states(m, v) == world       # the one exchange per mini-batch
        mn, vn = m.numpy(), v.numpy()
        w = (w - c[2] * mn / (np.sqrt(vn * c[3]) + c[4])).astype(np.float32)
        m = torch.from_numpy((mn * c[5] + mn * c[6]).astype(np.float32))
        v = torch.from_numpy((vn * c[7] + vn * c[8]).astype(np.float32))
    np.savez(Path(out_dir) / f"rank{rank}.npz", w=w, m=m.numpy(), v=v.numpy())
    dist.destroy_process_group()


def test_two_ranks_equal_one_device_with_NR_micro_batches(tmp_path):
    world, n, N, steps = 2, 64, 3, 3
    port = _free_port()
    mp.spawn(_rank_main, args=(world, port, n, N, steps, str(tmp_path)), nprocs=world, join=True)
    rng = np.random.default_rng(123)
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = rng.normal(0, 1e-2, (steps, world, N, n)).astype(np.float32)
    orc = AdamAOracle(w0.astype(np.float64), B1, B2, EPS)
    for step in range(steps):
        orc.begin_minibatch(N * world)
        for r in range(world):
            for i in range(N):
                # each rank scales by its local N, then the states are averaged over R ranks
                orc.fold(grads[step, r, i].astype(np.float64))
        orc.update(LR)
    res = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    for r in range(world):
        assert rel_l2(res[r]["w"], orc.theta) <= 1e-6
        assert rel_l2(res[r]["m"], B1 * orc.m) <= 1e-6
        assert rel_l2(res[r]["v"], world * B2 * orc.v) <= 1e-6      # pre-scaled for the next step
    assert np.array_equal(res[0]["w"], res[1]["w"])


def _sharded_rank_main(rank, world, port, n, N, steps, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(321)
    w = torch.from_numpy(rng.normal(0, 0.02, n).astype(np.float32))
    grads = rng.normal(0, 1e-2, (steps, world, N, n)).astype(np.float32)
    m = torch.zeros(n)
    v = torch.zeros(n)
    f = np.float32

    class NumpyApply:                      # stands in for the CUDA kernel, same constants
        def __init__(self):
            self.t = 0

        def apply_sharded(self, ws, ms, vs, lr, R):
            c = [f(x) for x in adama.host_constants(B1, B2, EPS, N, self.t, lr, world_size=R,
                                                    sharded=True)]
            mn, vn = ms.numpy().copy(), vs.numpy().copy()
            ws.copy_(torch.from_numpy((ws.numpy() - c[2] * mn / (np.sqrt(vn * c[3]) + c[4])).astype(f)))
            ms.copy_(torch.from_numpy((mn * c[5] + mn * c[6]).astype(f)))
            vs.copy_(torch.from_numpy((vn * c[7] + vn * c[8]).astype(f)))

    opt = NumpyApply()
    for step in range(steps):
        opt.t = step + 1
        a, b = [f(x) for x in adama.host_constants(B1, B2, EPS, N, opt.t, LR)[:2]]
        for i in range(N):
            g = grads[step, rank, i]
            m += torch.from_numpy(a * g)
            v += torch.from_numpy((b * g) * g)
        ddp.reduce_scatter_apply_allgather(opt, w, m, v, LR)
    lo, hi = ddp.shard_bounds(n, world, rank)
    np.savez(Path(out_dir) / f"shard{rank}.npz", w=w.numpy(), m=m.numpy(), v=v.numpy(), lo=lo, hi=hi)
    dist.destroy_process_group()


def test_sharded_states_two_ranks_equal_one_device(tmp_path):
    """Reduce-scatter, owner-only update with un-normalised storage, zeroed foreign shards,
    all-gather of w: same weights as one device with N*R micro-batches, and each rank keeps
    persistent state only for its own shard."""
    world, n, N, steps = 2, 64, 2, 3
    port = _free_port()
    mp.spawn(_sharded_rank_main, args=(world, port, n, N, steps, str(tmp_path)), nprocs=world,
             join=True)
    rng = np.random.default_rng(321)
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = rng.normal(0, 1e-2, (steps, world, N, n)).astype(np.float32)
    orc = AdamAOracle(w0.astype(np.float64), B1, B2, EPS)
    for step in range(steps):
        orc.begin_minibatch(N * world)
        for r in range(world):
            for i in range(N):
                orc.fold(grads[step, r, i].astype(np.float64))
        orc.update(LR)
    for r in range(world):
        d = np.load(tmp_path / f"shard{r}.npz")
        lo, hi = int(d["lo"]), int(d["hi"])
        assert rel_l2(d["w"], orc.theta) <= 1e-6                       # full weights everywhere
        assert rel_l2(d["m"][lo:hi], world * B1 * orc.m[lo:hi]) <= 1e-6
        assert rel_l2(d["v"][lo:hi], world ** 2 * B2 * orc.v[lo:hi]) <= 1e-6
        other = np.ones(n, bool)
        other[lo:hi] = False
        assert not d["m"][other].any() and not d["v"][other].any()


def test_bench_reference_arm_under_torchrun_prints_one_line():
    """Multi-rank launch contract: rank 0 alone runs and prints, the others exit 0."""
    port = _free_port()
    env = dict(os.environ, OMP_NUM_THREADS="2")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
         "--master-addr", "127.0.0.1", "--master-port", str(port), str(ROOT / "bench.py"),
         "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
        capture_output=True, text=True, timeout=600, env=env, cwd=str(ROOT))
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"


def _peer_states_rank(rank, world, port, out_dir):
    """PeerMappedStates with stand-ins for torch's symmetric memory (CPU tensors, made-up peer
    addresses) and for the optimizer: what is checked is the protocol around the one fused
    launch -- padding rule, zeroed accumulators, barrier / launch / barrier order, this rank's
    index and every rank's w, m, v addresses handed to adama_apply_sharded_peers."""
    import types
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log = []

    class Handle:
        def __init__(self, t, tag):
            self.buffer_ptrs = [1000 * tag + q for q in range(world)]
            self.tag = tag

        def barrier(self):
            dist.barrier()
            log.append(("barrier", self.tag))

    made = []

    def empty(n, dtype, device):
        t = torch.full((n,), 7.0, dtype=dtype)
        made.append(t)
        return t

    fake = types.ModuleType("torch.distributed._symmetric_memory")
    fake.empty = empty
    fake.rendezvous = lambda t, group: Handle(t, len(made))
    sys.modules["torch.distributed._symmetric_memory"] = fake
    torch.distributed._symmetric_memory = fake

    class Opt:
        def apply_sharded_peers(self, w_ptrs, m_ptrs, v_ptrs, r, n, lr):
            log.append(("launch", list(w_ptrs), list(m_ptrs), list(v_ptrs), r, n, lr))

    ok = True
    try:
        ddp.PeerMappedStates(4 * world + 4, "cpu")     # not a multiple of 4 * world
        ok = False
    except ValueError:
        pass
    n = 8 * world
    st = ddp.PeerMappedStates(n, "cpu")
    ok = ok and st.world == world and st.rank == rank and st.n == n
    ok = ok and bool((st.m == 0).all()) and bool((st.v == 0).all()) and bool((st.w == 7).all())
    st.exchange_and_apply(Opt(), 1e-3)
    kinds = [e[0] for e in log]
    ok = ok and kinds == ["barrier", "launch", "barrier"]
    launch = log[1]
    ok = ok and launch[4] == rank and launch[5] == n and launch[6] == 1e-3
    ok = ok and all(len(p) == world for p in launch[1:4])
    ok = ok and len({tuple(launch[1]), tuple(launch[2]), tuple(launch[3])}) == 3
    (Path(out_dir) / f"peer{rank}.json").write_text(json.dumps({"ok": bool(ok), "log": kinds}))
    dist.destroy_process_group()


def test_peer_mapped_states_protocol_with_stand_in_handles(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_peer_states_rank, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        res = json.loads((tmp_path / f"peer{r}.json").read_text())
        assert res["ok"], res
