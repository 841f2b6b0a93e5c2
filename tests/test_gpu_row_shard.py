"""Spatial sharding on the GPU path: `shard.RowShardedStep` splits every map by rows over 2 and 3 ranks and runs
the CUDA library on each rank's slab, with the boundary rows exchanged at the group inputs (forward) and the
overlapping input deltas added at their owners (backward).  One GPU is all there is here, so the ranks are
threads of one process on the same device (`shard.ThreadTransport`: queues between host threads; the launches
of all ranks are serialised on the stream and no kernel waits for another).  The sharded step must agree with
the untiled fp64 oracle, and with the one-GPU step, on the last map, the loss, the input gradient, the summed
filter gradient and the updated parameters.  Dyadic data: both precisions take the same discrete decisions."""
import numpy as np
import pytest
import torch

import paper_2409_09083_b200 as ftp
from paper_2409_09083_b200 import shard, synth
from _util import FP32_TOL, rel_err, run_gpu_step, run_oracle

WL = synth.with_slope(synth.Workload("y8", tuple(synth.stack_yolo8()), 2, 3, 96, 64, (1, 1), ((1, 2), (3, 4), (5, 8))), 0.5)


@pytest.mark.gpu
@pytest.mark.parametrize("world", [2, 3])
def test_row_sharded_step_matches_the_oracle_and_the_one_gpu_step(world):
    wl = WL
    x, params, target = synth.draw_dyadic(wl)
    lr = 0.25
    ref = run_oracle(wl, x, params, target=target, lr=lr)
    one = run_gpu_step(wl.with_(grid=(world, 1)), x, params, target, lr)
    rows = [s[1] for s in synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)]

    def rank_body(tr):
        xd, td = torch.from_numpy(x).cuda(), torch.from_numpy(target).cuda()
        pd = torch.from_numpy(params.copy()).cuda()
        st = shard.RowShardedStep(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.groups, tr)
        loss = st.step(xd, td, pd, lr)
        torch.cuda.synchronize()
        return dict(loss=loss, y=(st.y_lo, st.y_owned), dx=(st.dx_lo, st.dx_needed), grad=st.grad.cpu().numpy(),
                    params=pd.cpu().numpy(), needed=[t["needed_in"][tr.rank] for t in st.tables])

    out = shard.run_threads(world, rank_body)
    y = shard.gather_rows([o["y"] for o in out], rows[-1])
    dx = shard.gather_rows([o["dx"] for o in out], rows[0], add=True)
    # the exchange really happened: every rank needs rows it does not own at the inner group inputs
    assert all(o["needed"][1][1] - o["needed"][1][0] + 1 > rows[2] // world for o in out)
    assert np.array_equal(y, ref["y"])                                  # dyadic data: exact in any summation order
    for o in out:
        assert o["loss"] == pytest.approx(ref["loss"], rel=1e-5)
        assert rel_err(o["grad"], ref["dparams"]) <= FP32_TOL
        assert rel_err(o["params"], ref["new_params"]) <= FP32_TOL
        assert np.array_equal(o["grad"], out[0]["grad"])                # every rank holds the same sum
    assert rel_err(dx, ref["dx"]) <= FP32_TOL
    # ... and the one-GPU step with the same (world x 1) tile grid
    assert rel_err(out[0]["params"], one["new_params"]) <= 1e-5
    assert out[0]["loss"] == pytest.approx(one["loss"], rel=1e-5)
