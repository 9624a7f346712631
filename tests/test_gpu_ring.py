"""The ring all-reduce's data-plane step (libra_ring_step) on one GPU: R virtual ranks whose buffers live on the same
device, every step one launch per rank with the arrival flag already set (so no kernel ever waits for another kernel),
bit-exact against the oracle; the flag set by the host while the kernel polls; and the wait that runs out."""
import threading
import time

import numpy as np
import pytest

from oracle import ring_oracle as R

pytestmark = pytest.mark.gpu


def run_ring(lib, xs_dev, dtype, flag_ptr, status, elem_bytes, num_blocks=0):
    """Ring ReduceScatter + AllGather over the rows of xs_dev ([ranks, n] device tensor), in place."""
    import torch
    ranks, n = xs_dev.shape
    bounds = R.chunk_bounds(n, ranks)
    st = torch.cuda.current_stream().cuda_stream
    base = xs_dev.data_ptr()

    def ptr(r, c):
        return base + (r * n + bounds[c % ranks]) * elem_bytes

    def nbytes(c):
        return (bounds[c % ranks + 1] - bounds[c % ranks]) * elem_bytes

    for s in range(ranks - 1):
        for r in range(ranks):
            c, d = r - s, (r + 1) % ranks
            lib.libra_ring_step(0, ptr(d, c), ptr(d, c), ptr(r, c), nbytes(c), dtype, flag_ptr, 1, 1000000,
                                status.data_ptr(), num_blocks, st)
    for s in range(ranks - 1):
        for r in range(ranks):
            c, d = r + 1 - s, (r + 1) % ranks
            lib.libra_ring_step(0, ptr(d, c), 0, ptr(r, c), nbytes(c), dtype, flag_ptr, 1, 1000000,
                                status.data_ptr(), num_blocks, st)
    torch.cuda.synchronize()


@pytest.mark.parametrize("ranks,chunk", [(2, 4), (3, 4100), (4, 1 << 16), (8, 1028)])
def test_emulated_ring_is_bit_exact(lib, ranks, chunk):
    import torch
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(ranks)
    n = ranks * chunk
    flag = torch.ones(1, dtype=torch.int32, device=dev)
    status = torch.full((1,), 7, dtype=torch.int32, device=dev)
    # float32
    xs = [rng.standard_normal(n).astype(np.float32) * np.float32(10.0 ** rng.integers(-3, 4)) for _ in range(ranks)]
    want = R.ring_all_reduce(xs, "f32")
    d = torch.from_numpy(np.stack(xs)).to(dev)
    run_ring(lib, d, lib.RING_F32, flag.data_ptr(), status, 4, num_blocks=(0 if ranks != 4 else 5))
    got = d.cpu().numpy()
    assert int(status.item()) == 0
    for r in range(ranks):
        assert np.array_equal(got[r].view(np.uint32), want[r].view(np.uint32)), f"rank {r}"
    # bfloat16 (chunk boundaries stay multiples of 16 bytes: chunk % 8 == 0 or use 2 x chunk)
    n16 = ranks * chunk * 2
    xb = [torch.from_numpy(rng.standard_normal(n16).astype(np.float32)).to(torch.bfloat16) for _ in range(ranks)]
    wantb = R.ring_all_reduce([x.to(torch.float32).numpy() for x in xb], "bf16")
    db = torch.stack(xb).to(dev)
    run_ring(lib, db, lib.RING_BF16, flag.data_ptr(), status, 2)
    gotb = db.to(torch.float32).cpu().numpy()
    for r in range(ranks):
        assert np.array_equal(gotb[r], wantb[r]), f"bf16 rank {r}"


@pytest.mark.parametrize("ranks", [1, 2, 3, 4, 5, 6, 7, 8])
def test_library_schedule_over_local_buffers_is_bit_exact(lib, ranks):
    """libra_ring_all_reduce_local: the whole ReduceScatter + AllGather enqueued by the library from its own schedule
    records (pipeline pieces of a few KB here, so that every segment is several pieces), against the oracle."""
    import torch
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(40 + ranks)
    flag = torch.ones(1, dtype=torch.int32, device=dev)
    status = torch.full((1,), 7, dtype=torch.int32, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    for n_units, piece in ((ranks * 700 + 3, 4096), (max(1, ranks - 1), 16), (1 << 16, 16 << 20)):
        # float32: 4 elements per 16-byte unit
        n = n_units * 4
        xs = [rng.standard_normal(n).astype(np.float32) * np.float32(10.0 ** rng.integers(-3, 4)) for _ in range(ranks)]
        want = R.ring_all_reduce(xs, "f32", granule=4)
        bufs = [torch.from_numpy(x).to(dev) for x in xs]
        lib.libra_ring_all_reduce_local(0, [b.data_ptr() for b in bufs], n * 4, lib.RING_F32, piece, flag.data_ptr(), 1,
                                        1000000, status.data_ptr(), 0, st)
        torch.cuda.synchronize()
        assert ranks == 1 or int(status.item()) == 0
        for r in range(ranks):
            assert np.array_equal(bufs[r].cpu().numpy().view(np.uint32), want[r].view(np.uint32)), (n_units, piece, r)
        # bfloat16: 8 elements per unit
        n = n_units * 8
        xb = [torch.from_numpy(rng.standard_normal(n).astype(np.float32)).to(torch.bfloat16) for _ in range(ranks)]
        wantb = R.ring_all_reduce([x.to(torch.float32).numpy() for x in xb], "bf16", granule=8)
        bufs = [x.to(dev) for x in xb]
        lib.libra_ring_all_reduce_local(0, [b.data_ptr() for b in bufs], n * 2, lib.RING_BF16, piece, flag.data_ptr(), 1,
                                        1000000, status.data_ptr(), 3, st)
        torch.cuda.synchronize()
        for r in range(ranks):
            assert np.array_equal(bufs[r].to(torch.float32).cpu().numpy(), wantb[r]), (n_units, piece, r)
    with pytest.raises(lib.LibraError):
        lib.libra_ring_all_reduce_local(0, [bufs[0].data_ptr() + 4], 64, lib.RING_F32, 16, flag.data_ptr(), 1, 1000,
                                        status.data_ptr(), 0, st)


def test_flag_set_by_the_host_while_the_kernel_polls(lib):
    import torch
    dev = torch.device("cuda:0")
    n = 1 << 20
    own = torch.arange(n, dtype=torch.float32, device=dev)
    recv = torch.full((n,), 0.5, dtype=torch.float32, device=dev)
    dst = torch.zeros(n, dtype=torch.float32, device=dev)
    status = torch.full((1,), 7, dtype=torch.int32, device=dev)
    flag = torch.zeros(1, dtype=torch.int32).pin_memory()        # host-pinned, read by the kernel over the bus
    st = torch.cuda.current_stream().cuda_stream
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    lib.libra_ring_step(0, dst.data_ptr(), own.data_ptr(), recv.data_ptr(), n * 4, lib.RING_F32, flag.data_ptr(), 3,
                        5000000, status.data_ptr(), 2, st)

    def deliver():
        time.sleep(0.05)
        flag[0] = 2          # not yet: the step waits for 3
        time.sleep(0.05)
        flag[0] = 3

    th = threading.Thread(target=deliver)
    th.start()
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    th.join()
    assert int(status.item()) == 0
    assert 0.08 < waited < 3.0
    assert torch.equal(dst, own + 0.5)


def test_a_wait_that_runs_out_reports_and_leaves_the_context_usable(lib):
    import torch
    dev = torch.device("cuda:0")
    n = 4096
    own = torch.ones(n, dtype=torch.float32, device=dev)
    recv = torch.ones(n, dtype=torch.float32, device=dev)
    dst = torch.full((n,), -3.0, dtype=torch.float32, device=dev)
    status = torch.full((1,), 7, dtype=torch.int32, device=dev)
    flag = torch.zeros(1, dtype=torch.int32).pin_memory()        # nothing ever sets it
    st = torch.cuda.current_stream().cuda_stream
    t0 = time.perf_counter()
    lib.libra_ring_step(0, dst.data_ptr(), own.data_ptr(), recv.data_ptr(), n * 4, lib.RING_F32, flag.data_ptr(), 1,
                        200000, status.data_ptr(), 2, st)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert int(status.item()) == 1
    assert 0.15 < waited < 2.0
    assert torch.all(dst == -3.0)                                 # nothing was written
    flag[0] = 1
    lib.libra_ring_step(0, dst.data_ptr(), own.data_ptr(), recv.data_ptr(), n * 4, lib.RING_F32, flag.data_ptr(), 1,
                        200000, status.data_ptr(), 2, st)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.all(dst == 2.0)


def test_misuse_is_rejected(lib):
    import torch
    dev = torch.device("cuda:0")
    x = torch.zeros(64, dtype=torch.float32, device=dev)
    s = torch.zeros(1, dtype=torch.int32, device=dev)
    f = torch.ones(1, dtype=torch.int32, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    ok = dict(device=0, dst=x.data_ptr(), own=x.data_ptr(), recv=x.data_ptr(), nbytes=256, dtype=lib.RING_F32,
              flag=f.data_ptr(), expected=1, timeout=1000, status=s.data_ptr(), blocks=2)

    def call(**kw):
        a = dict(ok, **kw)
        lib.libra_ring_step(a["device"], a["dst"], a["own"], a["recv"], a["nbytes"], a["dtype"], a["flag"], a["expected"],
                            a["timeout"], a["status"], a["blocks"], st)

    call()
    for bad in (dict(nbytes=250), dict(dtype=5), dict(timeout=0), dict(timeout=20000000), dict(blocks=65),
                dict(dst=x.data_ptr() + 4), dict(recv=x.data_ptr() + 8), dict(device=-1)):
        with pytest.raises(lib.LibraError):
            call(**bad)
    torch.cuda.synchronize()
