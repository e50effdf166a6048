"""The allocation-free shield-row entry point against the workspace-based one.

`gelo_shield_rows_static` exists for callers that cannot allocate device memory (a plugin in
a process whose memory pool is owned by the host application, a runtime whose allocator is
frozen after start-up) and so cannot give the context a workspace.  It must produce exactly
what `gelo_shield_rows` produces.  The context used here has NO workspace, which also shows
that the call does not depend on one.  Two calls in a row check that what the first call
leaves in the shared built-in scratch does not leak into the second.

This file is named so that pytest collects it last.
"""
import pytest
import torch

from paper_2603_05035_b200 import binding, inputs

pytestmark = pytest.mark.gpu

TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_static_scratch_matches_workspace_variant(dt):
    ref_ctx = binding.Context(0)
    ref_ctx.ensure_workspace(4096, 204, 4096, 12288, dt)
    bare_ctx = binding.Context(0)                       # never given a workspace
    # two calls in a row with different sizes, so the second sees the first one's leftovers
    for n, d, k, seed in ((4096, 4096, 204, 5), (130, 256, 7, 6)):
        H = inputs.make_hidden(n, d, dt, seed, rms_norm=False, device="cuda")
        want = torch.full((k, d), float("nan"), device="cuda", dtype=TDT[dt])
        got = torch.full((k, d), float("nan"), device="cuda", dtype=TDT[dt])
        ref_ctx.shield_rows(H, n, d, k, 10.0, seed, dt, want)
        bare_ctx.shield_rows_static(H, n, d, k, 10.0, seed, dt, got)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        # same kernels, same arithmetic, same order: the bytes agree (well inside the stage
        # tolerances of 2e-6 / 4e-3 used for this step elsewhere)
        assert torch.equal(got, want)
    assert bare_ctx.last_status() == binding.OK
    ref_ctx.close(); bare_ctx.close()


def test_static_scratch_rejects_oversize_and_bad_arguments():
    ctx = binding.Context(0)
    L = binding.load_library()
    st = torch.cuda.current_stream().cuda_stream
    H = torch.zeros((8, 64), device="cuda"); S = torch.zeros((2, 64), device="cuda")
    too_many = 65536 + 1
    assert L.gelo_shield_rows_static(ctx._h, H.data_ptr(), too_many, 64, 2, 10.0, 0, 0, S.data_ptr(), st) == binding.ERR_UNSUPPORTED
    assert L.gelo_shield_rows_static(ctx._h, None, 8, 64, 2, 10.0, 0, 0, S.data_ptr(), st) == binding.ERR_INVALID
    assert L.gelo_shield_rows_static(ctx._h, H.data_ptr(), 8, 64, 2, 10.0, 0, 0, None, st) == binding.ERR_INVALID
    assert L.gelo_shield_rows_static(ctx._h, H.data_ptr(), 8, 60, 2, 10.0, 0, 0, S.data_ptr(), st) == binding.ERR_INVALID
    assert L.gelo_shield_rows_static(ctx._h, H.data_ptr(), 8, 64, 0, 10.0, 0, 0, None, st) == binding.OK
    ctx.close()
