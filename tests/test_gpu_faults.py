"""Error paths, injected from the host: every one must come back as an error code or a
completion status, with the pool untouched and the GPU context still usable."""
import numpy as np
import pytest
import torch

from paper_2605_03375_b200 import tutti as T
from paper_2605_03375_b200 import workload as wl
from tests.devcase import DeviceCase

pytestmark = pytest.mark.gpu


def small():
    return wl.config(2, 0.03, n_layers=2)


def test_bad_arguments():
    dc = DeviceCase(small())
    try:
        lib = dc.ctx.lib
        rc, *_ = dc.ring.tutti_build_sqes(dc.batch, 5, T.OP_READ, allow=(T.EINVAL,))
        assert rc == T.EINVAL                                    # layer out of range
        rc, *_ = dc.ring.tutti_build_sqes(dc.batch, 0, 9, allow=(T.EINVAL,))
        assert rc == T.EINVAL                                    # unknown opcode
        assert dc.ring.tutti_kv_restore_layer(1234, 1, allow=(T.EINVAL,)) == T.EINVAL
        rc, cqe = dc.ring.tutti_ring_poll(77)
        assert rc == T.EINVAL                                    # never reserved
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        rc2, cqe = dc.ring.tutti_ring_poll(first)
        assert rc2 == T.EAGAIN                                   # built but not issued
        assert dc.ring.tutti_kv_save_layer(first, n, allow=(T.EINVAL,)) == T.EINVAL  # READ IOCB
        dc.ring.tutti_kv_restore_layer(first, n)
        assert dc.poll_all(first, n)[0][1] == 0
        assert lib.tutti_pool_register(dc.ctx.h, 0, 8, 16, 32768, 4) == T.EINVAL     # misaligned
        assert lib.tutti_store_register(dc.ctx.h, 0, 4096, 16, 0) == T.EINVAL        # too small
        assert lib.tutti_set_option(dc.ctx.h, 99, 1) == T.EINVAL
        assert lib.tutti_set_option(dc.ctx.h, T.OPT_POOL_LAYOUT, 2) == T.EINVAL
    finally:
        dc.close()


def test_ring_full_then_drains():
    dc = DeviceCase(small(), depth=2)
    try:
        a = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        b = dc.ring.tutti_build_sqes(dc.batch, 1, T.OP_READ)
        rc, *_ = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ, allow=(T.EAGAIN,))
        assert rc == T.EAGAIN
        dc.ring.tutti_kv_restore_layer(a[1], a[2])
        dc.poll_all(a[1], a[2])
        c = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)     # room again
        assert c[0] == T.OK and c[1] == b[1] + b[2]
        dc.ring.tutti_kv_restore_layer(b[1], b[2])
        dc.ring.tutti_kv_restore_layer(c[1], c[2])
        dc.poll_all(b[1], b[2])
        dc.poll_all(c[1], c[2])
    finally:
        dc.close()


@pytest.mark.parametrize("what", ["block_id_high", "block_id_negative", "slot", "hit_unaligned",
                                  "short_row"])
def test_bad_batch_contents_reported_in_cqe(what):
    w = small()
    dc = DeviceCase(w)
    try:
        hit, ostart, oslot, bstart, bids = [t.clone() for t in dc.tensors]
        want = T.EFAULT
        if what == "block_id_high":
            bids[17] = w.n_pool_blocks
        elif what == "block_id_negative":
            bids[3] = -1
        elif what == "slot":
            oslot[1] = w.n_slots
        elif what == "hit_unaligned":
            hit[0] = hit[0] - 3
            want = T.EINVAL
        elif what == "short_row":
            hit[0] = hit[0] + 16 * 400
            want = T.EINVAL
        batch = T.make_batch(hit, ostart, oslot, bstart, bids)
        before = dc.pool_dev[0].clone()
        rc, first, n = dc.ring.tutti_build_sqes(batch, 0, T.OP_READ)
        info, _ = dc.ring.tutti_ring_read_iocb(first)
        assert info.status == want and info.total_entries == 0
        dc.ring.tutti_kv_restore_layer(first, n)
        cqes = dc.poll_all(first, n)
        assert all(c[1] == want and c[2] == 0 for c in cqes)
        assert torch.equal(dc.pool_dev[0], before)               # nothing was written
        # the ring and the context keep working
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        dc.ring.tutti_kv_restore_layer(first, n)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        assert np.array_equal(dc.pool_dev[0].cpu().numpy(), dc.oracle_restore(0))
    finally:
        dc.close()


@pytest.mark.parametrize("engine", [T.ENGINE_LDST, T.ENGINE_BULK])
def test_unpublished_iocb_times_out(engine):
    """An IOCB that was reserved but never filled: the kernel's bounded wait runs out, the
    completion carries TUTTI_ETIMEDOUT, and the next transfer works."""
    dc = DeviceCase(small())
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
        dc.ctx.tutti_set_option(T.OPT_WAIT_NS, 200_000)
        rc, first = dc.ring.tutti_ring_reserve(1, 16)
        before = dc.pool_dev[0].clone()
        dc.ring.tutti_kv_restore_layer(first, 1)
        (idx, status, nbytes), = dc.poll_all(first, 1)
        assert (idx, status, nbytes) == (first, T.ETIMEDOUT, 0)
        assert torch.equal(dc.pool_dev[0], before)
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        dc.ring.tutti_kv_restore_layer(first, n)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
    finally:
        dc.close()


def test_head_major_needs_16_byte_rows():
    """Rows of 8 bytes cannot be transposed in 16-byte vectors: the option is refused instead
    of producing misaligned accesses."""
    w = wl.make_workload("rows8", seed=3, n_layers=1, hit_tokens=[8], block_tokens=4, obj_tokens=8,
                         n_kv_heads=8, head_dim=8, elem_bytes=1, n_pool_blocks=16)
    dc = DeviceCase(w)
    try:
        assert dc.ctx.lib.tutti_set_option(dc.ctx.h, T.OPT_POOL_LAYOUT, T.POOL_HND) == T.EINVAL
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)      # still token-major
        dc.ring.tutti_kv_restore_layer(first, n)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        assert np.array_equal(dc.pool_dev[0].cpu().numpy(), dc.oracle_restore(0))
    finally:
        dc.close()


def test_bad_slot_in_a_large_batch_is_reported():
    """More than 8192 items: the keys are computed by a wide kernel; a slot out of range found
    there must still reach the completion status (and not poison the next build)."""
    w = wl.config(2, 0.6, n_layers=1, obj_tokens=16, slot_mean_run=2.0)
    assert 2 * len(w.obj_slot) > 8192
    dc = DeviceCase(w, depth=32, capacity=2048)
    try:
        hit, ostart, oslot, bstart, bids = [t.clone() for t in dc.tensors]
        oslot[len(oslot) // 2] = w.n_slots + 5
        bad = T.make_batch(hit, ostart, oslot, bstart, bids)
        rc, first, n = dc.ring.tutti_build_sqes(bad, 0, T.OP_READ)
        dc.ring.tutti_kv_restore_layer(first, n)
        cqes = dc.poll_all(first, n)
        assert all(c[1] == T.EFAULT and c[2] == 0 for c in cqes)
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        dc.ring.tutti_kv_restore_layer(first, n)
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        assert np.array_equal(dc.pool_dev[0].cpu().numpy(), dc.oracle_restore(0))
    finally:
        dc.close()


def test_bulk_stage_wait_running_out_still_completes_every_iocb():
    """The bulk engine's wait for a stage's bytes is made to report "ran out" from the host
    (TUTTI_OPT_INJECT_BULK_TIMEOUT; nothing on the GPU faults or hangs).  Every IOCB of the
    launch must still complete — with TUTTI_ETIMEDOUT — so that a poll never waits for ever,
    and the ring must keep working afterwards."""
    w = wl.config(2, 0.05, n_layers=3)
    dc = DeviceCase(w, depth=16, capacity=8, sgl_capacity=2 * len(w.block_ids) * 4)
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, T.ENGINE_BULK)
        for sm_count in (0, 8):
            dc.ctx.tutti_set_option(T.OPT_INJECT_BULK_TIMEOUT, 1)
            rc, first, per = dc.ring.tutti_build_sqes_layers(dc.batch, 0, 2, T.OP_READ)
            assert per > 1                                          # several IOCBs per layer
            infos = [dc.ring.tutti_ring_read_iocb(i)[0] for i in range(first, first + 2 * per)]
            dc.ring.tutti_kv_restore_layer(first, 2 * per, sm_count)
            cqes = dc.poll_all(first, 2 * per)
            assert sorted(c[0] for c in cqes) == list(range(first, first + 2 * per))
            for (idx, status, nbytes), info in zip(sorted(cqes), infos):
                if info.total_entries:
                    assert status == T.ETIMEDOUT, (idx, status)
                else:
                    assert status == 0 and nbytes == 0               # the empty tail of the reservation
            # stream waits on those IOCBs are released too (they completed, with an error)
            s2 = torch.cuda.Stream()
            rc2, f2, n2 = dc.ring.tutti_build_sqes(dc.batch, 2, T.OP_READ)
            dc.ring.tutti_kv_restore_layer(f2, n2, sm_count)
            dc.ring.tutti_stream_wait_iocb(f2, s2)
            s2.synchronize()
            dc.poll_all(f2, n2)
            # back to normal: the same ring moves the bytes
            dc.ctx.tutti_set_option(T.OPT_INJECT_BULK_TIMEOUT, 0)
            for layer in (0, 1):
                dc.pool_dev[layer].copy_(torch.from_numpy(dc.pool_host[layer]))
                rc, f, n = dc.ring.tutti_build_sqes(dc.batch, layer, T.OP_READ)
                dc.ring.tutti_kv_restore_layer(f, n, sm_count)
                assert all(c[1] == 0 for c in dc.poll_all(f, n))
                assert np.array_equal(dc.pool_dev[layer].cpu().numpy(), dc.oracle_restore(layer))
    finally:
        dc.close()


def test_stream_wait_refuses_an_iocb_that_was_not_issued():
    """A stream wait is enqueued only for an IOCB whose copy launch is already in the stream:
    for a built-but-unissued index the call answers TUTTI_EAGAIN and enqueues nothing (the
    stream stays free), so no stream can be left waiting for a completion nobody produces."""
    dc = DeviceCase(small())
    s_use = torch.cuda.Stream()
    try:
        rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, T.OP_READ)
        assert dc.ring.tutti_stream_wait_iocb(first, s_use, allow=(T.EAGAIN,)) == T.EAGAIN
        rc, rsv = dc.ring.tutti_ring_reserve(1, 16)                 # reserved, never filled
        assert dc.ring.tutti_stream_wait_iocb(rsv, s_use, allow=(T.EAGAIN,)) == T.EAGAIN
        done = torch.zeros(1, device=dc.dev)
        with torch.cuda.stream(s_use):
            done.add_(1)                                            # runs at once: nothing is waited for
        s_use.synchronize()
        assert done.item() == 1
        dc.ring.tutti_kv_restore_layer(first, n)
        assert dc.ring.tutti_stream_wait_iocb(first, s_use) == T.OK  # issued: accepted
        s_use.synchronize()
        assert all(c[1] == 0 for c in dc.poll_all(first, n))
        # the reserved IOCB is completed by a launch whose bounded wait runs out
        dc.ctx.tutti_set_option(T.OPT_WAIT_NS, 100_000)
        dc.ring.tutti_kv_restore_layer(rsv, 1)
        assert dc.poll_all(rsv, 1)[0][1] == T.ETIMEDOUT
    finally:
        dc.close()


@pytest.mark.parametrize("engine", [T.ENGINE_LDST, T.ENGINE_BULK])
@pytest.mark.parametrize("sm_count", [4, 8, 32])
def test_capped_launch_stays_on_sm_count_sms(engine, sm_count):
    """SM-capped mode on a plain stream (no green-context partition): the launch is exactly
    sm_count CTAs and they sit on sm_count different SMs, with either copy engine."""
    w = wl.config(2, 0.1, n_layers=1)
    dc = DeviceCase(w)
    try:
        dc.ctx.tutti_set_option(T.OPT_COPY_ENGINE, engine)
        for op in (T.OP_READ, T.OP_WRITE):
            rc, first, n = dc.ring.tutti_build_sqes(dc.batch, 0, op)
            (dc.ring.tutti_kv_restore_layer if op == T.OP_READ else dc.ring.tutti_kv_save_layer)(
                first, n, sm_count)
            assert all(c[1] == 0 for c in dc.poll_all(first, n))
            smids = dc.ring.tutti_ring_last_launch_sms()
            assert len(smids) == sm_count
            assert len(set(smids.tolist())) == sm_count
        assert np.array_equal(dc.pool_dev[0].cpu().numpy(), dc.oracle_restore(0))
    finally:
        dc.close()
