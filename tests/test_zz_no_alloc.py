"""based_prefill_static_scratch: the prefill entry point for callers that cannot allocate.

Collected last on purpose (the file name sorts after the others).  Through the C ABI, on a
shape whose sequence is split into segments (so the scratch is really used), the result is
compared with based_prefill's, twice in a row with different inputs: the second call finds
the first call's leftovers in the shared array and must not be affected by them.
"""
import pytest
import torch

import paper_2402_18668_b200 as based
from paper_2402_18668_b200 import workloads as wl
from parity import TOL_BF16, head_err, row_err

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_variant_twice():
    B, H, L, d_v = 2, 4, 16500, 64                      # 8 heads x 129 chunks -> 8 segments per head, state pass
    assert based.based_prefill_workspace_bytes(B, H, L, 16, d_v, based.BASED_BF16) > 0
    for seed in (21, 22):
        w = wl.Workload("noalloc", B, H, L, 16, d_v, "bf16", 0.25)
        q, k, v = (t.cuda() for t in wl.prefill_inputs(w, wl.generator(seed)))
        kv_ref, z_ref = based.new_state(B, H, d_v)
        ref = based.based_prefill(q, k, v, kv_state=kv_ref, z_state=z_ref)
        kv, z = based.new_state(B, H, d_v)
        out = torch.full_like(v, float("nan"))
        based.based_prefill_static_scratch(q, k, v, out, kv_state=kv, z_state=z)
        assert based.based_poll_error() == based.BASED_OK
        f64 = wl.to_f64
        assert row_err(f64(out), f64(ref)) <= TOL_BF16
        assert head_err(f64(kv), f64(kv_ref)) <= TOL_BF16
        assert head_err(f64(z), f64(z_ref)) <= TOL_BF16


def test_static_scratch_rejects_oversized_requests():
    B, H, L, d_v = 1, 18, 16384, 128                    # 7 partial states x 18 heads x 82,560 B > 8 MiB
    need = based.based_prefill_workspace_bytes(B, H, L, 16, d_v, based.BASED_BF16)
    assert need > based.based_static_scratch_bytes() == 8 << 20
    q = torch.zeros(B, H, L, 16, dtype=torch.bfloat16, device="cuda")
    v = torch.zeros(B, H, L, d_v, dtype=torch.bfloat16, device="cuda")
    n0 = based.launch_count()
    with pytest.raises(based.BasedError) as e:
        based.based_prefill_static_scratch(q, q.clone(), v, torch.empty_like(v))
    assert e.value.status == 6 and based.launch_count() == n0
