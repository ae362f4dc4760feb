"""The exchange step of vocabulary-parallel scoring on CPU: two gloo ranks each make the partials of
their shard (with the oracle, in the library's layout), all-gather them through the package's own
gather_partials, and merge; both must reproduce the unsharded log-probabilities."""
import json
import os
import socket
import subprocess
import sys

import numpy as np

from paper_2506_15733_b200 import vocab_parallel as VP

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = r"""
import json, math, sys
import numpy as np, torch
sys.path.insert(0, {root!r})
from oracle import specs_oracle as O
from oracle import specs_variants as V
from paper_2506_15733_b200 import inputs as I
from paper_2506_15733_b200 import vocab_parallel as VP
from paper_2506_15733_b200.replicas import Replicas
r = Replicas.from_env()
r.init("gloo")
cfg = I.StepConfig("vp", 7200, 1, 3, (5, 9), 32, 700, 0.3)
x = I.make_step_inputs(cfg)
v0, v1 = VP.shard_bounds(700, r.world, r.rank)
p = V.shard_partials(x.hidden, x.w_vocab, x.token_ids, v0, v1)
# the library's layout: base-2 maximum, sum of 2^(.), natural logit, pad
local = np.stack([p[:, 0] / math.log(2.0), p[:, 1], p[:, 2], np.zeros(len(p))], axis=1).astype(np.float32)
allp = VP.gather_partials(torch.from_numpy(local), r.world).numpy().astype(np.float64)
nat = np.stack([allp[:, :, 0] * math.log(2.0), allp[:, :, 1], allp[:, :, 2]], axis=2)
merged = V.merge_partials(nat, x.token_ids, 700)
whole = O.token_logprobs(x.hidden, x.w_vocab, x.token_ids)
print(json.dumps({{"rank": r.rank, "bounds": [v0, v1], "shape": list(allp.shape), "err": float(np.abs(merged - whole).max())}}))
r.shutdown()
"""


def test_shard_bounds_partition_the_vocabulary():
    for V, world in [(151936, 8), (152064, 3), (700, 2), (5000, 3), (100, 4), (256, 1)]:
        b = [VP.shard_bounds(V, world, r) for r in range(world)]
        assert b[0][0] == 0 and b[-1][1] == V and all(x[1] == y[0] for x, y in zip(b, b[1:]))
        assert all(lo % 256 == 0 for lo, _ in b)              # shards start on a vocabulary-tile boundary
        sizes = [hi - lo for lo, hi in b]
        assert max(sizes) - min(s for s in sizes[:-1] + [max(sizes)]) <= 256 or world > -(-V // 256)


def test_two_gloo_ranks_reproduce_the_unsharded_logprobs():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", RANK_SCRIPT.format(root=ROOT)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert [p.returncode for p in procs] == [0, 0], outs
    lines = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    assert lines[0]["bounds"][1] == lines[1]["bounds"][0] or lines[1]["bounds"][1] == lines[0]["bounds"][0]
    for l in lines:
        assert l["shape"][0] == 2 and l["shape"][2] == 4
        assert l["err"] < 1e-5                                 # fp32 partials on the wire
