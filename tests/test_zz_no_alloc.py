"""The workspace-free encode entry point (tahq_encode_noalloc), called through the C ABI.

It exists for callers that cannot allocate device memory themselves; its scratch is a fixed buffer
inside the library.  The packed bytes must equal those of tahq_encode, call after call (the buffer
is shared and keeps old contents, so the second call checks that everything that must start at zero
is cleared again).  This file is named to be collected last."""
import pytest
import torch

from paper_2506_01352_b200 import binding as T
from paper_2506_01352_b200 import synth


def _encode_noalloc(p, x):
    packed = torch.full((T.packed_bound(p),), 0x5A, dtype=torch.uint8, device=x.device)
    rc = T.tahq_encode_noalloc(p, x.data_ptr(), packed.data_ptr(), packed.numel(),
                               int(torch.cuda.current_stream().cuda_stream))
    assert rc == T.OK, T.status_string(rc)
    return packed


@pytest.mark.gpu
def test_noalloc_encode_matches_encode_on_two_calls_in_a_row():
    xa = synth.make("c2_gpt2s", device="cuda")                    # fp32, 8 ranking groups, direct selection
    xb = synth.make("c3_llama7b", device="cuda")                  # bf16, histogram selection
    pa = T.params_for(xa, group_tokens=1024, tile=64, budget_millibits=3800)
    pb = T.params_for(xb, group_tokens=2048, tile=64, budget_millibits=3500)
    assert T.workspace_bound(pa) <= T.NOALLOC_SCRATCH_BYTES and T.workspace_bound(pb) <= T.NOALLOC_SCRATCH_BYTES
    want_a = T.encode(pa, xa)
    want_b = T.encode(pb, xb)
    got_b1 = _encode_noalloc(pb, xb)          # first call on this device also looks up the scratch address
    got_a = _encode_noalloc(pa, xa)           # another configuration reuses the same scratch
    got_b2 = _encode_noalloc(pb, xb)          # and again: stale contents must not leak into the result
    torch.cuda.synchronize()
    assert torch.equal(got_b1, want_b)
    assert torch.equal(got_a, want_a)
    assert torch.equal(got_b2, want_b)
    y = T.decode(pb, got_b2)
    torch.cuda.synchronize()
    rel = ((y.float() - xb.float()).double().pow(2).sum() / xb.float().double().pow(2).sum()).item()
    assert rel < 0.05


def test_noalloc_encode_rejects_tensors_beyond_its_scratch():
    big = T.Params(tokens=65536, hidden=8192, dtype=T.BF16, group_tokens=4096, tile=64, budget_millibits=3800)
    assert T.workspace_bound(big) > T.NOALLOC_SCRATCH_BYTES
    # refused before any pointer is looked at and before anything is enqueued
    assert T.tahq_encode_noalloc(big, 4096, 8192, 1 << 40, 0) == T.ERR_TOO_LARGE
    assert "scratch" in T.status_string(T.ERR_TOO_LARGE)
