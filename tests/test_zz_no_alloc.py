"""nm_encoder_layer_static: the encoder layer for callers that cannot allocate device memory
(a framework's pool owns the GPU, a serving loop that must not call cudaMalloc, a plug-in that is
handed only its input and output).  Its scratch is a fixed array inside the library.  The test
drives it through the C ABI and checks it against nm_encoder_layer with a caller workspace, on
two calls in a row (the array keeps the previous call's contents), checks that the device's free
memory is the same before and after the calls (nothing was allocated), and checks the size limit.
Collected last on purpose: a failure here must not hide any other test."""
import numpy as np
import pytest
import torch

import nm_inputs
from util import BF16_ATOL, BF16_RTOL

pytestmark = pytest.mark.gpu


def test_static_scratch_layer_matches_workspace_layer(nm):
    from paper_2305_14405_b200.harness import EncoderModel
    ctx = nm.Context(0)
    try:
        cfg = nm_inputs.with_(nm_inputs.C2, B=2)          # 4.3 MB of scratch, well inside the 32 MiB array
        ctx.load_encoder_tables(cfg.segments, cfg.ranges())
        _, layers = nm_inputs.encoder_inputs(cfg, seed=3, random_affine=True)
        model = EncoderModel(ctx, cfg, layers)
        assert ctx.encoder_workspace_bytes(model.ccfg) <= nm.STATIC_WS_BYTES
        for call, seed in enumerate((11, 12)):             # two calls in a row, different inputs
            x_np = nm_inputs.matrix((cfg.T, cfg.H), seed, "bf16", 1.0)
            x = torch.from_numpy(x_np).cuda().bfloat16()
            want = model.forward_layer(0, x)               # existing entry point, caller workspace
            got = torch.full_like(x, float("nan"))
            torch.cuda.synchronize()
            free_before, _ = torch.cuda.mem_get_info()
            ctx.encoder_layer_static(model.structs[0], model.ccfg, x, got)
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            # the first call included: the array was placed when the context was created
            assert free_after == free_before, "call %d changed the device's free memory by %d bytes" % (
                call, free_before - free_after)
            ctx.check_device_status()
            g, w = got.float().cpu().numpy(), want.float().cpu().numpy()
            assert np.all(np.isfinite(g))
            assert np.all(np.abs(g - w) <= BF16_ATOL + BF16_RTOL * np.abs(w)), "call %d" % call
            assert torch.equal(got, want), "call %d: same kernels, same inputs, different scratch only" % call
        # a layer whose scratch exceeds the fixed array is refused with NM_ERR_WORKSPACE
        big = nm.Context.encoder_cfg(32, 512, 768, 12, 3072, nm.BF16)
        assert ctx.encoder_workspace_bytes(big) > nm.STATIC_WS_BYTES
        with pytest.raises(nm.NmError) as ei:
            ctx.encoder_layer_static(model.structs[0], big, x, got)
        assert ei.value.code == 8
    finally:
        ctx.close()
