"""CPU-side checks: the shared library loads and exports every symbol the header declares; the
multi-GPU host logic (request partition, reductions) works across two gloo ranks."""
import os
import re
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hvd.h")).read()
    return sorted(set(re.findall(r"HVD_API\s+[\w\s\*]+?\b(hvd_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2606_01019_b200 as H
    lib = H.load_library()
    names = declared_symbols()
    assert len(names) >= 9 and "hvd_verify_commit" in names and "hvd_lookup" in names
    for n in names:
        assert getattr(lib, n) is not None
    assert names == H.exported_symbols()           # the binding covers the whole header
    assert lib.hvd_status_string(0) == b"HVD_OK" and lib.hvd_status_string(3) == b"HVD_ERR_UNSUPPORTED"


def test_binding_structs_have_the_layout_of_the_header(tmp_path):
    """The ctypes mirrors of the header's structs (sizes and the offset of every field) against what a C
    compiler makes of include/hvd.h."""
    import ctypes as C
    from paper_2606_01019_b200 import binding as b
    pairs = [("hvd_config", b.HvdConfig), ("hvd_host_step_args", b.HvdHostStepArgs), ("hvd_next_cycle", b.NextCycle)]
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "hvd.h"', 'int main(void) {']
    for cname, cls in pairs:
        lines.append(f'  printf("{cname} %zu", sizeof({cname}));')
        for field, _ in cls._fields_:
            lines.append(f'  printf(" %zu", offsetof({cname}, {field}));')
        lines.append('  printf("\\n");')
    lines += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.strip().splitlines()
    assert len(out) == len(pairs)
    for line, (cname, cls) in zip(out, pairs):
        got = line.split()
        want = [cname, str(C.sizeof(cls))] + [str(getattr(cls, f).offset) for f, _ in cls._fields_]
        assert got == want, (cname, got, want)


def test_no_cpu_fallback_without_a_device():
    import torch
    import pytest
    import paper_2606_01019_b200 as H
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(H.HvdError):
        H.Context(max_batch=4, k_cap=8, max_hist_len=100, max_rows=36, max_vocab=100)


def test_product_code_never_touches_the_oracle():
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2606_01019_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower().replace("no cpu or pytorch fallback", ""), f


def test_partition_requests():
    from paper_2606_01019_b200.sharding import partition_requests, request_cost
    rng = np.random.default_rng(0)
    for B, world in [(64, 2), (64, 8), (512, 4), (3, 8), (1, 2), (7, 7)]:
        cost = request_cost(rng.integers(512, 65536, B), rng.integers(4, 33, B), 128256, 2)
        b = partition_requests(cost, world)
        assert b[0] == 0 and b[-1] == B and (np.diff(b) >= 0).all()
        if B >= 4 * world:
            per = np.array([cost[b[r]:b[r + 1]].sum() for r in range(world)])
            assert per.max() <= per.mean() + cost.max()          # balanced to within one request
    b = partition_requests(np.ones(8), 2)
    assert list(b) == [0, 4, 8]


_RANK_PROGRAM = r"""
import os, sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from paper_2606_01019_b200.sharding import max_over_ranks, sum_over_ranks, partition_requests, request_cost
import hvd_workloads as W
from oracle import pipeline as P
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = W.CONFIGS["C1"].scaled(B=6)
inp = P.prepare(w)
bounds = partition_requests(request_cost(inp.rq.hist_len, inp.rq.K, w.V, w.elt), world)
lo, hi = int(bounds[rank]), int(bounds[rank + 1])
# each rank steps only its own requests (here with the CPU oracle standing in for the device)
sub = W.subset_requests(inp.rq, lo, hi)
rows = slice(int(inp.rq.row_off[lo]), int(inp.rq.row_off[hi]))
part = P.Inputs(w, sub, inp.W1, inp.b1, inp.W2, inp.b2, inp.tau, A=inp.A[lo:hi], strict=inp.strict[lo:hi], logits_np=inp.logits_np[rows])
out = P.step(part, sub.copy())
full = P.step(inp, inp.rq.copy())
assert (out.vf.accepted == full.vf.accepted[lo:hi]).all() and (out.vf.committed == full.vf.committed[lo:hi]).all()
tokens = sum_over_ranks(float(out.vf.n_commit.sum()))
assert tokens == float(full.vf.n_commit.sum()), (tokens, full.vf.n_commit.sum())
assert max_over_ranks(10.0 + rank) == 10.0 + world - 1
dist.destroy_process_group()
sys.stdout.write("rank %d ok %d %d\n" % (rank, lo, hi))
"""


def test_two_gloo_ranks_shard_requests_and_reduce(tmp_path):
    prog = tmp_path / "rank_program.py"
    prog.write_text(_RANK_PROGRAM.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29631", str(prog)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "rank 0 ok" in res.stdout and "rank 1 ok" in res.stdout


_KEYS_PROGRAM = r"""
import sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from paper_2606_01019_b200.sharding import reduce_keys_over_ranks, vocab_shards
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
rng = np.random.default_rng(7)                       # the same rows on every rank
rows, V = 40, 1001
x = rng.normal(0, 1, (rows, V)).astype(np.float32)
x[3, [5, 700]] = 9.0                                 # equal maxima in different shards: the lower index wins
x[4, [900, 901]] = 9.0                               # and inside one shard
x[5] = -3.0                                          # a constant negative row
x[6, 10] = 0.0; x[6, 600] = -0.0; x[6, np.arange(V) % 590 != 10] = -1.0   # +0 and -0 are equal
b = vocab_shards(V, world)
lo, hi = int(b[rank]), int(b[rank + 1])
def keys_of(shard, offset):
    # what the header promises of a key: larger logit first, then the lower global index; signed order
    u = shard.view(np.uint32).astype(np.uint64)
    u = np.where((u << np.uint64(33)) == 0, np.uint64(0), u)                 # -0 -> +0
    o = np.where(u >> np.uint64(31) == 1, (~u) & np.uint64(0xffffffff), u | np.uint64(0x80000000))
    idx = np.arange(shard.shape[1], dtype=np.uint64) + np.uint64(offset)
    k = (o << np.uint64(32)) | ((~idx) & np.uint64(0xffffffff))
    best = k.max(axis=1)
    return (best ^ np.uint64(1 << 63)).view(np.int64)
keys = torch.from_numpy(keys_of(x[:, lo:hi], lo).copy())
keys[7] = torch.iinfo(torch.int64).min if rank == 0 else keys[7]             # a row one rank did not read
reduce_keys_over_ranks(keys)
got = (~(keys.numpy().view(np.uint64) & np.uint64(0xffffffff))) & np.uint64(0xffffffff)
want = np.array([int(np.argmax(np.where(r == 0, 0.0, r))) for r in x])
if world > 1 and lo <= want[7] < hi and rank == 0:
    pass
ok = [i for i in range(rows) if i != 7]
assert (got[ok].astype(np.int64) == want[ok]).all(), (got, want)
assert got[3] == 5 and got[4] == 900 and got[5] == 0 and got[6] == 10
dist.destroy_process_group()
sys.stdout.write("rank %d keys ok\n" % rank)
"""


def test_two_gloo_ranks_reduce_vocabulary_shard_keys(tmp_path):
    prog = tmp_path / "keys_program.py"
    prog.write_text(_KEYS_PROGRAM.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29633", str(prog)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "rank 0 keys ok" in res.stdout and "rank 1 keys ok" in res.stdout
