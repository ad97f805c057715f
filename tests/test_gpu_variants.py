"""GPU: the ways the library can schedule one and the same training step give the same bits.

The switches of csrc/env.hpp are read once per process, so every variant runs in a process of its
own (a few lines of Python that print a digest of every output); the digests must agree.  Covered:
the backward run kernel with groups of batch rows and the clustered one without, the input projections a window
ahead on their own stream or in the step's stream, the step on a stream of urgent priority, and no
overlap at all.
"""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import hashlib, json, sys
import numpy as np
sys.path.insert(0, {root!r})
from paper_1606_03401_b200 import harness, synth
cfg = synth.with_overrides(synth.CONFIGS["c2"], input=128, hidden=256, batch=64, readout=96, t=70)
dp = harness.DeviceProblem(cfg, want_dx=True)
out = {{}}
for name, plan in (("msm", dp.plan("msm", 7)), ("full", dp.full_memory_plan())):
    res = dp.run(plan)
    assert res["counters"][3] == 0, res["counters"]
    h = hashlib.sha256()
    for k in sorted(res):
        if k in ("counters",) or res[k] is None:
            continue
        h.update(k.encode())
        h.update(np.ascontiguousarray(res[k]).tobytes() if hasattr(res[k], "tobytes") else repr(res[k]).encode())
    out[name] = h.hexdigest()
    out[name + "_fwd_ops"] = int(res["counters"][0])
print("DIGEST " + json.dumps(out))
"""


def digest(env_extra):
    env = dict(os.environ)
    for k in ("MEBPTT_NO_BWD_GROUPS", "MEBPTT_NO_ZX_AHEAD", "MEBPTT_PRIORITY", "MEBPTT_NO_OVERLAP", "MEBPTT_BWD_CLUSTER"):
        env.pop(k, None)
    env.update(env_extra)
    out = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT)], env=env, capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("DIGEST ")][-1]
    return json.loads(line[len("DIGEST "):])


def test_scheduling_variants_give_the_same_bits():
    base = digest({})
    assert base["msm"] == base["full"]                      # the plan does not change a bit either
    # (the clustered backward kernel without groups, at the groups' cluster size: the partial sums
    # of a column are then added in the same order)
    for env in ({"MEBPTT_BWD_CLUSTER": "4"}, {"MEBPTT_NO_ZX_AHEAD": "1"}, {"MEBPTT_PRIORITY": "1"},
                {"MEBPTT_NO_OVERLAP": "1"}):
        assert digest(env) == base, env
