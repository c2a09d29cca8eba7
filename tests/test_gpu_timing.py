"""Optional per-call timing (App. D path classification: D2D and H2D gather times of a switch;
Sec. 3.3 measured restore cost): CUDA-event times of the last offload / restore / stage."""
import numpy as np
import pytest
import torch

from paper_2607_17181_b200 import binding as tb
from paper_2607_17181_b200 import workloads as wl
from tests.gpu_util import DevicePool, GuardedPinned

pytestmark = pytest.mark.gpu


def test_timing_of_offload_restore_and_stage_legs():
    ctx = tb.Talaria(0, bounce_bytes=4 << 20, dma_min_bytes=1 << 20)
    try:
        with pytest.raises(tb.TalariaError) as e:
            ctx.get_timing()                                          # nothing has been timed yet
        assert e.value.status == tb.ERR_INVALID_ARG
        shape, nb, n = wl.TINY, 256, 200
        pool = DevicePool(shape, wl.kv_pool(wl.rng(730), shape, nb))
        img = GuardedPinned(n * shape.bytes_per_block)
        hl = tb.host_layout(wl.dense_strides(shape, n, "PF"), img.n)
        table = np.arange(n, dtype=np.int32)
        ctx.kv_offload(pool.kv, table, 0, n, img.ptr, hl)             # timing is off by default
        ctx.sync()
        with pytest.raises(tb.TalariaError):
            ctx.get_timing()
        ctx.set_timing(True)
        for variant_n in (n, 2):                                      # copy-engine variant, then the zero-copy kernel
            ctx.kv_offload(pool.kv, table, 0, variant_n, img.ptr, hl)
            t = ctx.get_timing()                                      # waits for the call
            assert t.op == 1 and t.total_ms > 0 and t.d2h_ms == t.total_ms and t.h2d_ms == 0 and t.d2d_ms == 0
            ctx.kv_restore(pool.kv, table[::-1].copy(), 0, variant_n, img.ptr, hl)
            t = ctx.get_timing()
            assert t.op == 2 and t.total_ms > 0 and t.h2d_ms == t.total_ms and t.d2h_ms == 0
        # a switch with clean and dirty chunks: both legs are timed, on the streams they run on
        nbytes, chunk = 64 << 20, 2 << 20
        staging = torch.randint(0, 255, (nbytes,), dtype=torch.uint8, device="cuda")
        slots = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        host = torch.randint(0, 255, (nbytes,), dtype=torch.uint8).pin_memory()
        plan = np.zeros(nbytes // chunk, tb.COPY_DTYPE)
        for k in range(plan.size):
            plan[k] = (staging.data_ptr() + k * chunk, host.data_ptr() + k * chunk, slots.data_ptr() + k * chunk, chunk, k, 0)
        dirty = np.zeros((plan.size + 7) // 8, np.uint8)
        dirty[0] = 0b1010
        for run in ("stage", "prepared"):
            if run == "stage":
                ctx.stage(plan, dirty)
            else:
                prepared = ctx.stage_plan_create(plan)
                ctx.stage_plan_run(prepared, dirty)
            t = ctx.get_timing()
            assert t.op == 3 and t.d2d_ms > 0 and t.h2d_ms > 0 and t.d2h_ms == 0
            assert t.total_ms >= 0.9 * max(t.d2d_ms, t.h2d_ms)
        ctx.stage(plan, None)                                         # all clean: no host leg
        t = ctx.get_timing()
        assert t.op == 3 and t.d2d_ms > 0 and t.h2d_ms == 0
        ctx.stage_plan_destroy(prepared)
        ctx.sync()
        want = staging.clone()
        assert torch.equal(slots, want)
        # a match from host memory: first copy to last kernel, both forms
        g = wl.rng(731)
        sess = wl.tokens(g, 5000)
        cont = wl.continuation(g, sess, 5200, 4000)
        res = np.zeros(1, tb.MATCH_DTYPE)
        out_h = np.zeros(5200 // 16, np.uint64)
        ctx.prefix_match_host(1, cont, [0, cont.size], sess, [0, sess.size], None, 16, wl.HASH_SEED, out_h, res)
        t = ctx.get_timing()
        assert t.op == 4 and 0 < t.total_ms < 5000 and t.d2d_ms == 0 and t.h2d_ms == 0 and t.d2h_ms == 0
        d_tokens = torch.zeros(16384, dtype=torch.int32, device="cuda")
        d_hashes = torch.zeros(1024, dtype=torch.int64, device="cuda")
        ctx.stage(plan, None)
        ctx.prefix_match_resident([(sess, 0, 0, 8192, 0, -1)], d_tokens, d_hashes, 16, wl.HASH_SEED, res)
        assert ctx.get_timing().op == 4
        ctx.prefix_match_resident([(cont, 8192, 512, 0, sess.size, 0)], d_tokens, d_hashes, 16, wl.HASH_SEED, res)
        t = ctx.get_timing()
        assert t.op == 4 and 0 < t.total_ms < 5000 and int(res[0]["lcp_tokens"]) == 4000
        ctx.set_timing(False)
        ctx.kv_offload(pool.kv, table, 0, 2, img.ptr, hl)
        ctx.sync()
        assert ctx.get_timing().op == 4                               # untouched by calls made with timing off
    finally:
        ctx.destroy()
