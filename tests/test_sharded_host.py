"""Group-per-device mapping (paper_1905_10395_b200/sharded.py), host logic on CPU: the split of the groups, the
cross-rank election rule, and the exchange protocol itself -- in one process and under torch.distributed with
2 gloo ranks -- with a CPU stand-in for the device engine.  The sharded run must equal the single-population
oracle bit for bit."""
import itertools
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs, sharded
from tests._shard_cpu_engine import CpuShardEngine, argmin_by_rule, pack_key

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_partition_covers_every_group_once():
    for G, world in [(1, 1), (4, 2), (5, 2), (7, 3), (8, 8)]:
        parts = sharded.partition_groups(G, world)
        assert [g for p in parts for g in p] == list(range(G))
        assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
    with pytest.raises(ValueError):
        sharded.partition_groups(2, 3)


def test_cross_rank_election_rule_equals_the_election_on_the_whole_population():
    # every rank packs its best (loss, global index) into a key; the minimum key must be the global argmin with
    # the same treatment of ties, signed zeros, infinities and NaN
    vals = [-np.inf, -1.0, -0.0, 0.0, 1.0, np.inf, np.nan]
    for combo in itertools.product(vals, repeat=4):
        loss = np.array(combo, dtype=np.float32)
        group_of = np.array([0, 0, 1, 1], dtype=np.int32)
        ll, gl = orc.elect(loss, group_of, 2)
        keys = []
        for r, idx in enumerate(([0, 1], [2, 3])):
            p = argmin_by_rule(loss[idx], idx)
            assert idx[p] == ll[r]                       # the local pick is the local leader
            keys.append(pack_key(loss[idx[p]], idx[p]))
        assert (min(keys) & 0xFFFFFFFF) == gl, (combo, keys, gl)


def test_packed_keys_order_like_the_election_rule():
    vals = [-np.inf, -3.5, -1e-30, -0.0, 0.0, 1e-30, 2.0, np.inf, np.nan]
    for a in vals:
        for b in vals:
            for ia, ib in ((1, 2), (2, 1)):
                want = argmin_by_rule([a, b], [ia, ib])
                got = 0 if pack_key(a, ia) < pack_key(b, ib) else 1
                assert got == want, (a, b, ia, ib)


@pytest.mark.parametrize("world", [1, 2, 3])
def test_lockstep_exchange_reproduces_the_single_population_bit_for_bit(world):
    steps = 11
    rng = np.random.default_rng(3)
    group_of = np.sort(np.concatenate([np.arange(6), rng.integers(0, 6, 9)])).astype(np.int32)   # unequal groups
    w = inputs.make_external(15, 6, 257, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=3, steps=steps, loss_ring=4,
                             config_id=141, group_of=group_of)
    w.arrays["loss_ring"][2, :] = np.nan                 # an all-NaN election elects worker 0
    engines = [CpuShardEngine(w, r, world) for r in range(world)]
    sharded.run_lockstep(engines, steps)
    o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau)
    o.run(steps)
    for e in engines:
        assert np.array_equal(e.x_local().view(np.uint32), o.x[e.shard.workers].view(np.uint32))
        assert e.global_leader_global == o.gl
    ll = np.concatenate([e.local_leaders_global for e in engines])
    assert np.array_equal(ll, o.ll)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _json_objects(text):
    """Every JSON object in the ranks' joint output (two ranks may write on one line)."""
    dec, out, pos = json.JSONDecoder(), [], 0
    while True:
        pos = text.find("{", pos)
        if pos < 0:
            return out
        try:
            obj, end = dec.raw_decode(text, pos)
            out.append(obj)
            pos = end
        except json.JSONDecodeError:
            pos += 1


def test_two_gloo_ranks_exchange_the_global_leader():
    for attempt in range(2):                             # the probed port can be taken before the ranks bind it
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr",
               "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "tests", "_gloo_shard_worker.py")]
        r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
        if r.returncode == 0:
            break
    assert r.returncode == 0, r.stderr[-3000:]
    lines = _json_objects(r.stdout)
    assert sorted(l["rank"] for l in lines) == [0, 1]
    owners = set()
    for l in lines:
        assert l["rows_equal"], l
        assert l["leaders"] == l["want"], l
        owners.update(g for g in l["want"])
    # the run must have needed the exchange: global leaders owned by both ranks
    w0 = next(l["workers"] for l in lines if l["rank"] == 0)
    assert any(g in w0 for g in owners) and any(g not in w0 for g in owners)
