"""mala_decode_static -- the decode entry point for callers that cannot allocate device memory.

Such callers (a serving engine with a fixed memory plan, a plug-in that is handed nothing but its input and
output buffers, a path that must stay clear of the allocator) pass no workspace: the split partials live in
an array inside the library.  The test calls the entry point through the C ABI twice in a row on different
inputs -- the second call finds the first call's partials in the shared array -- and checks both results
against the oracle and, bit for bit, against mala_decode with caller-provided scratch, and that an over-sized problem
is refused without a launch.
Collected last so that a failure here cannot hide the other GPU tests."""
import numpy as np
import pytest
import torch

from paper_2609_32712_b200 import workloads as W
from tests import parity

pytestmark = pytest.mark.gpu


def test_decode_static_matches_decode_on_two_calls_in_a_row(oracle):
    from paper_2609_32712_b200 import mala
    tau = 1e-4
    outs = []
    for seed, (Nk, S, preset) in enumerate([(8192, 8, "D"), (5000, 16, "literal")]):
        w = W.custom_decode(2, 8, 2, Nk, 128, S, group_types=["diffuse", "peaked"], seed=20 + seed, preset=preset)
        q, kc, vc = (w[x].cuda() for x in ("q", "kcache", "vcache"))
        o_static, lse_static = mala.decode_static(q, kc, vc, w["scale"], tau, S)
        outs.append((w, q, kc, vc, S, o_static, lse_static))
    torch.cuda.synchronize()
    for (w, q, kc, vc, S, o_static, lse_static) in outs:
        # against the oracle, at the limits every decode test uses ...
        ref = oracle.decode(w["q"], w["kcache"], w["vcache"], w["scale"], tau, S, 128)
        parity.check_output(o_static.float().cpu().numpy()[:, 0], ref["o"])
        assert np.abs(lse_static.cpu().numpy() - ref["lse"]).max() <= parity.LSE_ABS
        # ... and bit for bit against mala_decode with caller-provided scratch: both run the same deterministic
        # kernels, so anything left over in the shared array that reached a result would show here
        o_ref, lse_ref, _ = mala.decode(q, kc, vc, w["scale"], tau, S)
        torch.cuda.synchronize()
        assert torch.equal(o_static, o_ref)
        assert torch.equal(lse_static, lse_ref)
    assert mala.device_status() == 0


def test_decode_static_refuses_problems_beyond_its_scratch():
    from paper_2609_32712_b200 import mala
    # 16 * 16 * 1024 splits * (128 + 1) floats = 135 MB of partials > 24 MiB
    B, Hq, Hkv, Nk, S = 16, 16, 1, 2048, 1024
    assert mala.workspace_bytes(mala.OP_DECODE, B, Hq, Hkv, Nk, 128, S) > mala.STATIC_SCRATCH_BYTES
    q = torch.zeros(B, 1, Hq, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(B, Nk, Hkv, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mala.MalaError) as e:
        mala.decode_static(q, kv, kv, 0.1, 1e-4, S)
    assert e.value.code == -9
