"""kvs_truncate: dropping the newest tokens and decoding the same steps again."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_2410_18517_b200 import KvsError
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild

from helpers import assert_close, make_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


@pytest.mark.parametrize("Hq,Hkv,dtype,context", [(4, 4, "bf16", 250), (8, 2, "bf16", 127), (4, 2, "f32", 64)])
@pytest.mark.parametrize("use_step", [False, True])
def test_steps_run_again_after_a_truncate_match_a_fresh_oracle(Hq, Hkv, dtype, context, use_step):
    """Five decode steps, cut back to the context, five steps with OTHER inputs: the second run must
    equal an oracle that never saw the first five tokens (stale rows past the cut are never read)."""
    w = si.Workload(f"trunc_{Hq}_{Hkv}_{dtype}_{context}", L=3, Hq=Hq, Hkv=Hkv, D=128, B=2, context=context,
                    dtype=dtype, n_shared=1, map_seed=0, steps=5, fixed_map=(0, 1, 0))
    sm = w.share_map()
    cache = make_cache(w, 5, sm)
    orc = oracle.Oracle(w.L, w.Hq, w.Hkv, w.D, w.B, sm)
    for l in range(w.L):
        k, v = si.context_kv(w, l)
        orc.layer_forward(l, None, k.double().numpy(), v.double().numpy())
        cache.append(l, k.cuda(), v.cuda())

    def steps(first, check):
        for t in range(first, first + 5):
            for l in range(w.L):
                q, k, v = si.step_qkv(w, t, l)
                own = sm[l] == l
                if use_step:
                    out = cache.decode_step(l, q.cuda(), k.cuda() if own else None, v.cuda() if own else None)
                else:
                    cache.append(l, k.cuda(), v.cuda())
                    out = cache.decode_attention(l, q.cuda())
                if check:
                    ref = orc.layer_forward(l, q.double().numpy(), k.double().numpy(), v.double().numpy())
                    assert_close(out.cpu().numpy(), ref, f"second run, step {t} layer {l}")

    steps(0, check=False)
    assert cache.seq_len(0) == context + 5
    cache.truncate(context)
    assert [cache.seq_len(l) for l in range(w.L)] == [context] * w.L
    steps(100, check=True)
    assert cache.seq_len(2) == context + 5 and cache.device_status() == 0
    # cutting to more rows than there are changes nothing; a negative count is refused
    cache.truncate(context + 50)
    assert cache.seq_len(0) == context + 5
    with pytest.raises(KvsError) as e:
        cache.truncate(-1)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG


def test_truncate_refuses_a_slot_rows_were_evicted_from():
    w = si.Workload("trunc_ragged", L=2, Hq=2, Hkv=2, D=64, B=1, context=40, dtype="bf16", n_shared=0, map_seed=0, steps=1)
    cache = make_cache(w, 2)
    for l in range(w.L):
        k, v = si.context_kv(w, l)
        cache.append(l, k.cuda(), v.cuda())
    keep = torch.arange(40, dtype=torch.int32).repeat(1, 2, 1).contiguous().cuda()
    cache.evict(1, keep, np.array([[30, 20]], dtype=np.int32))
    with pytest.raises(KvsError) as e:
        cache.truncate(10)
    assert e.value.status == kb.KVS_ERR_STATE
    assert cache.seq_len(0) == 40 and cache.seq_len(1) == 30      # nothing was changed
    cache.truncate(35)                                            # only the un-evicted slot is longer than 35
    assert cache.seq_len(0) == 35 and cache.seq_len(1) == 30
