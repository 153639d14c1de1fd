"""Full-size parity on sampled rows: the benchmark workloads in the launch configuration bench.py
times, checked against the oracle on a sample of rows the oracle computes one by one."""
import numpy as np
import pytest
import torch

from paper_2604_26209_b200 import synth
from tests.util import oracle_step, err_stats

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3


@pytest.fixture(scope="module")
def rt():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26209_b200 import runtime
    return runtime


@pytest.mark.parametrize("make,n_sample", [(lambda: synth.config_main(n_prompts=64), 96),
                                           (lambda: synth.config_long(n_prompts=32), 48)])
def test_fullsize_sampled_rows(rt, make, n_sample):
    s = make()
    tb = synth.make_tensors(s)
    rng = np.random.default_rng(123)
    rows = np.sort(rng.choice(s.n_active, size=n_sample, replace=False))
    # make sure first/last rows of documents and of the batch are in the sample
    rows[:4] = [0, 1, s.n_active - 2, s.n_active - 1]
    rows = np.unique(rows)
    meta, want = oracle_step(s, tb, rows=rows)
    db = rt.DeviceBatch(s, tb)
    db.build_meta()
    tabs = db.tables()
    assert tabs["n_active"] == s.n_active
    act = tabs["active_slot"][: s.n_active]
    db.set_step_inputs(tb["q"][act], tb["k_new"][act], tb["v_new"][act])
    db.rope()
    db.kv_append()
    db.attn(True)
    torch.cuda.synchronize()
    assert db.status() == 0
    o = synth.bf16_bits_to_f32(rt.bits_of(db.o))
    mx, mean = err_stats(o[rows], want.o)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)
    # properties that hold at any size: every written row is finite; rows beyond n_active untouched
    assert np.isfinite(o[: s.n_active]).all()
    lse = db.lse.cpu().numpy()[: s.n_active]
    assert np.max(np.abs(lse[rows] - want.lse)) <= 2e-2
