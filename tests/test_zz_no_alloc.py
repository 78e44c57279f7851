"""reflex_adarmsnorm_noalloc: the AdaRMSNorm entry point for callers that cannot allocate or lend scratch memory
(its gate scratch is an array built into the library). Checked through the C ABI against reflex_adarmsnorm with a
caller-provided gate_buf, on two calls in a row that share the built-in array, and against the CPU oracle (Eq. 2 with
non-zero gate biases). Collected last on purpose."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2607_14695_b200 import synth  # noqa: E402


def test_noalloc_matches_scratch_entry_point_twice():
    from paper_2607_14695_b200 import build as rbuild
    rbuild.build()
    from paper_2607_14695_b200 import binding as rb
    from oracle import reflex_oracle as orc
    import gpu_util as U
    dev = "cuda:0"
    up = lambda a, w: (torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(dev).to(rb.torch_dtype(w.dtype))).contiguous()
    # two different shapes back to back: the second call finds the first call's values in the shared array
    for w, t, variant in ((synth.CONFIGS["cfg4"], 0.3, 0), (synth.CONFIGS["cfg2"].with_(B=5), 0.9, 1), (synth.CONFIGS["cfg1"], 0.5, 2)):
        hx, hcond, hW = synth.norm_input(w, 0, variant), synth.cond_vectors(w, t), synth.gate_weights(w, variant, std=0.05, bias_std=0.2)
        want = orc.adarmsnorm_batched(hx, hcond, *hW, 1e-6)
        x, cond = up(hx, w), up(hcond, w)
        W1, b1, W2, b2 = [up(a, w) for a in hW]
        y_ref = torch.full_like(x, float("nan"))
        gate_buf = torch.empty((w.B * (w.D + w.Hd),), dtype=torch.float32, device=dev)
        rb.reflex_adarmsnorm(x, y_ref, cond, W1, b1, W2, b2, gate_buf=gate_buf)
        for _ in range(2):
            y = torch.full_like(x, float("nan"))
            rb.reflex_adarmsnorm_noalloc(x, y, cond, W1, b1, W2, b2)
            torch.cuda.synchronize()
            assert torch.isfinite(y.float()).all()
            # same kernels on the same inputs: the tolerance of the parity tests is met with room to spare (bitwise equal)
            assert (y.float() - y_ref.float()).abs().max().item() <= 2e-2
            assert torch.equal(y, y_ref)
            U.check_close(U.to_host(y), want, w.dtype, f"noalloc {w.name} vs oracle", rel_clause=True)
    # beyond the built-in scratch: refused with a clear message, nothing launched
    big = synth.CONFIGS["cfg4"].with_(B=128)
    xb = torch.zeros((big.B, 1, big.D), dtype=torch.bfloat16, device=dev)
    cb = torch.zeros((big.B, big.Cd), dtype=torch.bfloat16, device=dev)
    W1, b1, W2, b2 = [up(a, big) for a in synth.gate_weights(big, 0)]
    with pytest.raises(rb.ReflexError) as e:
        rb.reflex_adarmsnorm_noalloc(xb, torch.empty_like(xb), cb, W1, b1, W2, b2)
    assert e.value.code == rb.ERR_SHAPE and "exceeds the built-in scratch" in str(e.value)
