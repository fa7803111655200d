"""Host side of the whole-step launch: rwkvq_step_plan_bytes / rwkvq_step_plan_cover build the complete
schedule on the host (no GPU needed: device pointers are only stored), so shapes, ordering, argument
checks and the schedule's coverage are tested here."""
import ctypes as C

import numpy as np
import pytest

from paper_2505_03803_b200 import binding as B
from paper_2505_03803_b200 import build as build_mod
from paper_2505_03803_b200 import inputs


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def _desc(method, oc, ic, bits):
    if method == B.RWKVQ_SQ:
        return B.Desc(method=1, bits=3, oc=oc, ic=ic, group=128, vec_dim=1, tile=0, entries=0,
                      oc_pad=-(-oc // 128) * 128, ic_pad=-(-ic // 256) * 256, image_bytes=0, stream_bytes=0)
    return B.Desc(method=0, bits=bits, oc=oc, ic=ic, group=0, vec_dim=2, tile=256, entries=1 << bits, oc_pad=oc, ic_pad=ic,
                  image_bytes=0, stream_bytes=0)


def _mu_desc(ic, bits=6):
    return B.Desc(method=0, bits=bits, oc=1, ic=ic, group=0, vec_dim=2, tile=0, entries=1 << bits, oc_pad=1, ic_pad=ic,
                  image_bytes=0, stream_bytes=0)


def _ops(d, h, layers, vq_every=3, bits=6, y_dtype=B.RWKVQ_F32, one_stage=False):
    rows = []
    addr = 1 << 30
    for l in range(layers):
        for (name, oc, ic, has_mu, stage) in inputs.layer_shapes(d, h):
            rows.append((oc, ic, has_mu, 0 if one_stage else 4 * l + stage))
    rows.sort(key=lambda r: r[3])
    arr = (B.GemvOp * len(rows))()
    for k, (oc, ic, has_mu, stage) in enumerate(rows):
        o = arr[k]
        vq = vq_every > 0 and k % vq_every == 0 and oc % 256 == 0 and ic % 256 == 0
        o.W_desc = _desc(B.RWKVQ_VQ if vq else B.RWKVQ_SQ, oc, ic, bits)
        for field in ("W_image_dev", "x_fp16_dev", "y_dev"):
            setattr(o, field, addr)
            addr += 1 << 26
        if has_mu:
            o.mu_desc = _mu_desc(ic, bits)
            o.mu_image_dev = addr
            o.xprev_fp16_dev = addr + (1 << 20)
            addr += 1 << 26
        o.stage, o.y_dtype = stage, y_dtype
    return arr


@pytest.mark.parametrize("d,h,layers,Bn,bits", [(512, 1280, 2, 1, 6), (2048, 7168, 24, 1, 6), (4096, 14336, 4, 8, 6), (4096, 14336, 2, 16, 8)])
def test_plan_is_built_for_benchmark_shapes(d, h, layers, Bn, bits):
    ops = _ops(d, h, layers, bits=bits)
    n = B.rwkvq_step_plan_bytes(ops, Bn)
    assert n > 0 and n % 256 == 0
    # the plan grows with the number of units: twice the layers, roughly twice the descriptors
    n2 = B.rwkvq_step_plan_bytes(_ops(d, h, 2 * layers, bits=bits), Bn)
    assert 1.5 * n < n2 < 2.5 * n


# Every record (product, 16-row slice, 256-column tile) must reach exactly one consumer warp exactly
# once, in each of the planner's three ways of dealing a stage (row of tiles by row of tiles; whole
# units at their cost midpoints; eighths of a unit for stages too small for either): small and large
# stages, ragged shapes (rows that end in half a unit, ic not a multiple of 256), every batch
# regime, few and many CTAs, every product in one stage.
@pytest.mark.parametrize("d,h,layers,Bn,bits,n_ctas,one_stage", [
    (512, 1280, 2, 1, 6, 148, False),
    (384, 896, 2, 5, 6, 148, False),
    (2048, 7168, 2, 1, 6, 148, False),
    (4096, 14336, 1, 1, 6, 148, False),
    (4096, 14336, 1, 2, 6, 148, False),
    (4096, 14336, 1, 8, 6, 148, False),
    (4096, 14336, 1, 16, 8, 148, False),
    (4096, 14336, 1, 16, 8, 7, False),        # many slices per CTA: phases are cut to the warp count
    (2048, 7168, 3, 1, 6, 148, True),         # every product in one stage
    (2048, 7168, 1, 8, 6, 33, True),
    (512, 1280, 1, 12, 8, 16, False),
])
def test_schedule_covers_every_record_once(d, h, layers, Bn, bits, n_ctas, one_stage):
    ops = _ops(d, h, layers, bits=bits, one_stage=one_stage)
    counts, per_cta = B.rwkvq_step_plan_cover(ops, Bn, n_ctas)
    assert counts.size == sum((o.W_desc.oc // 16) * (o.W_desc.ic_pad // 256) for o in ops)
    assert (counts == 1).all(), f"{int((counts != 1).sum())} records not dealt exactly once"
    assert int(per_cta.sum()) == counts.size
    if n_ctas == 148 and not one_stage:
        # whole units (16 records of a 256-column tile) are dealt by cost: no CTA carries more than
        # its even share plus two units per stage
        n_stages = len({o.stage for o in ops})
        assert per_cta.max() <= counts.size / n_ctas + n_stages * 32


def test_plan_rejects_bad_arguments():
    ops = _ops(512, 1280, 1)
    assert B.rwkvq_step_plan_bytes(ops, 0) == 0 and B.rwkvq_step_plan_bytes(ops, 17) == 0
    assert B.rwkvq_step_plan_bytes(_ops(512, 1280, 1, y_dtype=B.RWKVQ_F16), 1) == 0      # the step writes fp32 outputs
    bad = _ops(512, 1280, 1)
    bad[2].stage = -1                                                                  # stages must not decrease
    assert B.rwkvq_step_plan_bytes(bad, 1) == 0
    bad = _ops(512, 1280, 1)
    bad[0].x_fp16_dev = bad[0].x_fp16_dev + 8                                          # 16-byte alignment
    assert B.rwkvq_step_plan_bytes(bad, 1) == 0
    bad = _ops(512, 1280, 1)
    bad[1].W_desc.ic = 200                                                             # shape the format does not support
    assert B.rwkvq_step_plan_bytes(bad, 1) == 0
    lib = B.lib()
    assert lib.rwkvq_step_run(None, 0, None) == 1
    assert lib.rwkvq_step_run(C.c_void_p(4096), 1 << 20, None) == 1                     # not a buffer a plan was written to
    assert lib.rwkvq_step_plan_release(C.c_void_p(4096)) == 1
    assert lib.rwkvq_step_set_wait(C.c_void_p(4096), 0, 0) == 1
    with pytest.raises(B.RwkvqError):
        B.rwkvq_step_plan_cover(_ops(512, 1280, 1), 0, 148)
