"""The kernels' bounded waits, made to run out on purpose -- without hanging, trapping or faulting anything.

Every wait of one thread block on another (grid barrier, descriptor and prefix polls, the decoder's queue of
large groups) has an iteration limit.  These tests shorten the limits (fastsgd_debug_set_wait_limits), put a
counter of the workspace where no block can ever complete it, and check that the launch ends by itself with
FASTSGD_ST_TIMEOUT in every status word, that nothing outside the output buffers was written, that the library
refuses further work until the workspace is registered again, and that it is exact again afterwards.
"""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import Guarded
from paper_2112_04291_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _streams_equal_oracle(grads, pg, po, outs):
    for g, o in zip(grads, outs):
        total, d, status = binding.stream_info(o)
        orc, ostream = oracle.compress(g, po)
        assert status == orc == 0 and total == ostream.size
        assert np.array_equal(o[:total].cpu().numpy(), ostream)


@pytest.mark.parametrize("n,workers", [(5_000_011, 3), (1_000_003, 1)])
def test_grid_barrier_that_cannot_complete_ends_in_timeout(n, workers):
    # 3 gradients of 306 tiles: two teams of blocks with their own barriers; 1 gradient: the single-gradient kernel
    host = [workloads.student_t_layers(n, seed=40 + w, blocks=9) for w in range(workers)]
    base = workloads.base_for_keep(host[0], n // 300)
    pg, po = binding.params(base), oracle.params(base)
    ws = binding.ensure_workspace(n, pg)
    grads = [torch.from_numpy(g).cuda() for g in host]
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    bufs = [Guarded(cap, fill=0x11) for _ in range(workers)]
    outs = [b.view for b in bufs]
    try:
        assert binding.compress_batch(grads, pg, outs) == 0
        _streams_equal_oracle(host, pg, po, outs)
        # gradient 0's barrier counter starts beyond reach: no block is ever the last to arrive, nobody sets the flag
        binding.debug_set_wait_limits(block_polls=4096, copy_tries=256)
        binding.workspace_u32("bar_count", 8)[0] = 0x40000000
        torch.cuda.synchronize()
        assert binding.compress_batch(grads, pg, outs) == 0          # the launch itself is accepted ...
        for o in outs:                                              # ... and ends by itself, every stream marked
            total, d, status = binding.stream_info(o)
            assert (total, d, status) == (64, 0, binding.ST_TIMEOUT)
        assert all(b.intact() for b in bufs)
        # the workspace's counters are not at rest: further work is refused until it is registered again
        assert binding.compress_batch(grads, pg, outs) == binding.E_NO_WORKSPACE
        dense = torch.zeros(n, dtype=torch.float32, device="cuda")
        assert binding.decompress_accumulate(outs[0], cap, n, pg, dense) == binding.E_NO_WORKSPACE
    finally:
        binding.debug_set_wait_limits(0, 0, 0)
        binding.set_workspace(ws)
    assert binding.compress_batch(grads, pg, outs) == 0
    _streams_equal_oracle(host, pg, po, outs)
    assert all(b.intact() for b in bufs)


def test_decoder_queue_slot_that_is_never_filled_ends_in_timeout():
    n = 5_000_011
    host = workloads.normal_outliers(n, seed=3)
    base = workloads.base_for_keep(host, n // 20)            # 5 %: every group is decoded by a whole block
    pg, po = binding.params(base), oracle.params(base)
    ws = binding.ensure_workspace(n, pg)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    out = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    assert binding.compress(torch.from_numpy(host).cuda(), pg, out) == 0
    orc, ostream = oracle.compress(host, po)
    odense = np.zeros(n, np.float32)
    assert orc == 0 and oracle.decompress_accumulate(ostream, n, po, odense) == 0
    buf = Guarded(4 * n)
    dense = buf.view.view(torch.float32)
    try:
        # five queue slots count as reserved although nothing will ever fill them: their takers' waits run out
        binding.debug_set_wait_limits(queue_polls=2000)
        binding.workspace_u32("queue_counters", 6)[4] = 5
        torch.cuda.synchronize()
        assert binding.decompress_accumulate(out, cap, n, pg, dense) == 0
        assert binding.decode_status() == binding.ST_TIMEOUT
        assert buf.intact()
        # the queue is back in its resting state all the same
        assert not bool(binding.workspace_u32("queue_counters", 6).any().item())
        assert not bool(binding.workspace_u32("queue_slots", 4096).any().item())
        assert binding.decompress_accumulate(out, cap, n, pg, dense) == binding.E_NO_WORKSPACE
    finally:
        binding.debug_set_wait_limits(0, 0, 0)
        binding.set_workspace(ws)
    dense.zero_()
    assert binding.decompress_accumulate(out, cap, n, pg, dense) == 0
    assert binding.decode_status() == 0
    assert np.array_equal(dense.cpu().numpy(), odense) and buf.intact()
