"""Parallelized deployment: the chunk update on one stream while decode runs on another with a
serving copy of the module; the new module is swapped in at a decode-step boundary."""
import numpy as np
import pytest
import torch

from oracle import templora_oracle as orc
from paper_2401_11504_b200 import inputs
from parity_utils import TOL, assert_close, f64, hp32, snapshot_block

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2401_11504_b200 import build
    build.build_library()
    from paper_2401_11504_b200 import binding
    binding.templora_set_kernel_path(0)
    return binding


@pytest.mark.parametrize("partition", [True, False])
def test_decode_sees_old_module_until_publish(b, partition):
    # partition=True: the two streams own disjoint groups of SMs; False: ordinary streams with per-stream caps
    from paper_2401_11504_b200 import runtime
    shapes = [("q", 512, 512), ("gate", 512, 1408), ("down", 1408, 512)]
    hp = hp32(dict(lr=2e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0))
    blk = runtime.Block(b, 3, "pardep", shapes, 512, 64, 2.0, "bf16", "cuda")
    snap = snapshot_block(blk)
    dep = runtime.ParallelDeployment(b, blk, n_tokens=4, update_sms=116, decode_sms=32, partition=partition)
    assert (dep.partition is not None) == partition
    try:
        xs = [f64(x) for x in dep.x]
        old = [orc.decode_fwd(x, p["W0"], p["A_master"], p["B_master"], 2.0) for x, p in zip(xs, snap)]
        dep.decode_step()
        torch.cuda.synchronize()
        first = [y.clone() for y in dep.y]
        for y, ref in zip(first, old):
            assert_close("decode before the update", f64(y), ref, TOL["bf16"])

        # the update runs while decode keeps stepping; decode must keep giving the old module's output
        dep.start_update(2, hp)
        for _ in range(6):
            dep.decode_step()
        dep.decode_stream.synchronize()
        for y, y0 in zip(dep.y, first):
            assert torch.equal(y, y0), "decode output changed before the module was published"

        dep.publish()
        dep.decode_step()
        torch.cuda.synchronize()
        assert b.templora_read_device_status(dep.ws_upd)[0] == 0
        assert b.templora_read_device_status(dep.ws_dec)[0] == 0
        ref, steps = orc.update_block(snap, 2, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"],
                                      bf16_work=True)
        assert steps == dep.step == 2
        changed = 0
        for i, (y, y0, x, p, q) in enumerate(zip(dep.y, first, xs, snap, ref)):
            # what decode must now compute: the device's own updated working copies
            A, Bm = f64(blk.state[i]["A"]["work"]), f64(blk.state[i]["B"]["work"])
            assert_close("decode after publish", f64(y), orc.decode_fwd(x, p["W0"], A, Bm, 2.0), TOL["bf16"])
            # and those working copies are the oracle's updated module (to the Adam step's conditioning)
            assert np.abs(A - orc.round_bf16(q["A_master"].astype(np.float32))).max() <= 4 * hp["lr"] + 1e-2 * np.abs(A).max()
            changed += int(not torch.equal(y, y0))
        assert changed == len(dep.y), "the published module did not change the decode output"
    finally:
        dep.close()


def test_stream_sm_limit_keeps_results(b):
    # a capped stream computes the same thing with fewer CTAs
    from parity_utils import check_fwd_bwd
    st = torch.cuda.Stream()
    b.templora_set_stream_sm_limit(st, 24)
    try:
        with torch.cuda.stream(st):
            check_fwd_bwd(b, 31, "capped", 300, 512, 640, 64, 2.0, "bf16")
    finally:
        b.templora_set_stream_sm_limit(st, 0)


def test_sm_partition_splits_the_device_and_both_streams_compute(b):
    # the two groups cover the device's SMs between them, each stream carries the matching cap, and a
    # forward/backward on either stream (tensors made on the default stream) matches the oracle
    from parity_utils import check_fwd_bwd
    total = torch.cuda.get_device_properties(0).multi_processor_count
    part = b.templora_sm_partition_create(32)
    try:
        assert part.sms_first >= 32 and part.sms_rest >= 1 and part.sms_first + part.sms_rest <= total
        assert part.sms_first % 8 == 0
        for handle, tag in ((part.stream_first, "part-first"), (part.stream_rest, "part-rest")):
            st = torch.cuda.ExternalStream(handle)
            torch.cuda.synchronize()
            with torch.cuda.stream(st):
                check_fwd_bwd(b, 33, tag, 300, 512, 640, 64, 2.0, "bf16")
            st.synchronize()
    finally:
        b.templora_sm_partition_destroy(part)
    assert part.handle is None
    with pytest.raises(b.TemploraError):
        b.templora_sm_partition_create(0)
    with pytest.raises(b.TemploraError):
        b.templora_sm_partition_create(total)
