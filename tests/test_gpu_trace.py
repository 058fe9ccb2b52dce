"""The tracing build (-DKVS_TRACE): the attention kernels stamp a per-block timeline that
`python -m paper_2410_18517_b200.timeline` turns into a report.  Run here on two small shapes (one that
needs the combine kernel, one whose units are finished inside the split-K kernel): the stamps must be
there for every block and in order, and the results must still be right (the script checks the status word;
the normal parity tests cover the arithmetic)."""
import json
import os
import subprocess
import sys

import pytest
import torch

from paper_2410_18517_b200 import KvsError, SharedKVCache
from paper_2410_18517_b200 import binding as kb

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("batch,context,combine", [(4, 700, True), (24, 300, False)])
def test_timeline_of_a_small_run(batch, context, combine):
    out = subprocess.run([sys.executable, "-m", "paper_2410_18517_b200.timeline", "--batch", str(batch), "--context",
                          str(context), "--layers", "2", "--steps", "3"], capture_output=True, text=True, timeout=900,
                         cwd=ROOT, env=dict(os.environ, PYTHONPATH=ROOT))
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-2000:]
    r = json.loads(out.stdout.strip().splitlines()[-1])
    assert r["launches_reported"] == 4 and (r["workload"]["combine_launches"] > 0) == combine
    # per block: entry <= wait returns <= first tile <= end, all within a millisecond of the launch's start
    for i in range(3):
        assert 0 <= r["entry"][i] <= r["consumer_wait_returns"][2] + 1e-6
    assert r["consumer_wait_returns"][0] <= r["first_tile"][0] <= r["end"][0]
    assert r["first_tile"][2] <= r["end"][2] <= 1000.0
    assert r["stream_us_median_block"] > 0 and r["pieces_per_block"] >= 1
    if combine:
        c = r["combine_last_block"]
        assert c[0] <= c[1] <= c[2] and c[1] >= r["end"][0]     # it waits for the split-K kernel, then runs
    else:
        assert "combine_last_block" not in r


def test_the_normal_build_refuses_to_trace():
    cache = SharedKVCache(1, 2, 2, 64, 1, 16, "bf16")
    buf = torch.zeros(160 * 32, dtype=torch.int64, device="cuda")
    with pytest.raises(KvsError) as e:
        kb.kvs_trace_begin(cache.ctx, buf, buf.numel() * 8)
    assert e.value.status == kb.KVS_ERR_STATE
    assert kb.kvs_trace_end(cache.ctx) == 0
