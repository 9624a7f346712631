"""The two read-ceiling entry points (measurement aids): they run, flag nothing, reject misuse, and leave the
handle in a state where the next real step is still correct."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [(8, 2, 128), (4, 1, 64), (32, 2, 128)])
def test_gather_read_then_real_step(lib, shape):
    import torch
    Hq, Hkv, d = shape
    dev = torch.device("cuda:0")
    lens = [700, 33, 0, 2049]
    lens_a, bt, q, k, v = W.random_case(91, len(lens), Hq, Hkv, d, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    r = H.Runner(lib, Hq, Hkv, d, k.shape[0], len(lens), bt.shape[1], plan=lib.PlanParams(4, 1, 2, 16, 16, 64))
    qd, kd, vd, btd = (H.to_dev(x, dev) for x in (q, k, v, bt))
    lens_dev = torch.from_numpy(lens_a).to(dev)
    st = torch.cuda.current_stream().cuda_stream
    junk = torch.zeros((len(lens), Hq, d), dtype=torch.int16, device=dev)
    with pytest.raises(lib.LibraError):   # no plan yet
        r.h.debug_gather_read(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                              junk.data_ptr(), st)
    r.h.plan(lens_a, r.ws.data_ptr(), r.ws.numel(), st)
    n0 = r.h.launch_count()
    for _ in range(2):
        r.h.debug_gather_read(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                              junk.data_ptr(), st)
    torch.cuda.synchronize()
    assert r.h.launch_count() == n0 + 2
    assert r.h.debug_error_word() == 0
    # the arrival counters were left clean: a real step on the same workspace gives the right answer
    got = H.bf16_dev_to_f32(r.run(qd, kd, vd, btd, lens_a))
    assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
    # the pools were only read
    assert np.array_equal(kd.cpu().numpy().view(np.uint16), k) and np.array_equal(vd.cpu().numpy().view(np.uint16), v)
    r.h.close()


def test_stream_read(lib):
    import torch
    dev = torch.device("cuda:0")
    lens_a, bt, q, k, v = W.random_case(92, 1, 4, 1, 64, [40])
    r = H.Runner(lib, 4, 1, 64, k.shape[0], 1, bt.shape[1])
    st = torch.cuda.current_stream().cuda_stream
    buf = torch.arange(1 << 20, dtype=torch.int32, device=dev)
    with pytest.raises(lib.LibraError):
        r.h.debug_stream_read(buf.data_ptr(), buf.numel() * 4, st)     # needs a planned workspace
    r.h.plan(lens_a, r.ws.data_ptr(), r.ws.numel(), st)
    for nbytes in (16, 48, 4096 + 16, buf.numel() * 4, buf.numel() * 4 - 5):
        r.h.debug_stream_read(buf.data_ptr(), nbytes, st)
    torch.cuda.synchronize()
    assert r.h.debug_error_word() == 0
    assert torch.equal(buf, torch.arange(1 << 20, dtype=torch.int32, device=dev))
    for bad in ((buf.data_ptr() + 4, 64), (buf.data_ptr(), 8), (0, 64)):
        with pytest.raises(lib.LibraError):
            r.h.debug_stream_read(bad[0], bad[1], st)
    r.h.close()
