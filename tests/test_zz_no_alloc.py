"""The workspace-free patch-merging entry point (mixaq_merge_forward_static) against the regular one.

Some users of the library run it where device memory cannot be allocated any more (inside an application whose
pool owns the device, in a frame loop that must not synchronise, under a no-allocation policy after start-up).
For them the merge has a variant whose intermediate sits in an array built into the library.  This file checks,
through the C ABI, that the variant returns exactly what mixaq_merge_forward returns, on two calls in a row that
share the built-in array (the second smaller than the first, so stale bytes of the first call lie behind it),
and that a problem beyond the array's size is refused with a clear message.  It is collected last on purpose.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_2507_19131_b200 import synth  # noqa: E402


@pytest.fixture(scope="module")
def mq():
    from paper_2507_19131_b200 import binding
    if not torch.cuda.is_available():
        pytest.fail("GPU test selected but no CUDA device is visible")
    return binding


def test_static_merge_matches_the_workspace_merge_on_two_calls_in_a_row(mq):
    ctx = mq.Context(0)
    try:
        cases = [(96, 2, 41, 57, 8), (64, 1, 9, 11, 4)]          # (C, B, H, W, activation bits); odd sizes pad
        prepared = []
        for (Cc, B, H, W, bits) in cases:
            m = synth.make_merge(np.random.default_rng(Cc + bits), Cc, 4, bits)
            x = torch.from_numpy(synth.input_blobs(Cc + 7, B, H, W, Cc, bg_std=0.5)).cuda()
            dm = mq.DeviceMerge(ctx, m)
            want = mq.merge_forward(ctx, dm, x)
            y = torch.full_like(want, float("nan"))               # the caller's output buffer
            prepared.append((dm, x, want, y))
        torch.cuda.synchronize()
        for dm, x, want, y in prepared:                            # two calls back to back on one stream
            mq.merge_forward_static(ctx, dm, x, y)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        for dm, x, want, y in prepared:
            got, ref = y.cpu().numpy(), want.cpu().numpy()
            scale = max(float(np.abs(ref).max()), 1e-30)
            assert float(np.abs(got - ref).max()) <= 1e-3 * scale
            assert np.array_equal(got, ref)
    finally:
        ctx.close()


def test_static_merge_refuses_what_does_not_fit(mq):
    ctx = mq.Context(0)
    try:
        Cc, B, H, W = 96, 4, 200, 334                            # 4*100*167 rows x 384 bytes = 25.6 MB > 8 MiB
        m = synth.make_merge(np.random.default_rng(3), Cc, 4, 8)
        dm = mq.DeviceMerge(ctx, m)
        x = torch.zeros((B, H, W, Cc), device="cuda")
        y = torch.zeros((B, (H + 1) // 2, (W + 1) // 2, 2 * Cc), device="cuda")
        assert B * 100 * 167 * 4 * Cc > mq.STATIC_SCRATCH_BYTES
        with pytest.raises(mq.MixaqError) as e:
            mq.merge_forward_static(ctx, dm, x, y)
        assert e.value.status == -3
        assert "built-in scratch holds" in str(e.value)
        assert ctx.device_status() == 0
    finally:
        ctx.close()
