"""The append entry point that brings its own scratch (``lagkv_compress_append_noalloc``).

Some users of this library run where no device memory can be had at call time: inside a
serving engine whose pool is fully handed out, in a callback on somebody else's stream, or
under a policy that forbids ``cudaMalloc`` after start-up.  They cannot supply the workspace
``lagkv_compress_append`` asks for, so the library keeps a fixed 1 MiB array of its own and
this entry point uses it.  The checks here: through the C ABI, on two calls in a row (the
array is shared and keeps the previous call's contents), the result is identical to the
workspace-taking entry point's -- caches, lengths and kept positions bit for bit, which is
the bar the other append tests use -- and to the float64 oracle's replay of the same append;
a request beyond the array's size is refused.

This file sorts last on purpose: a run that stops at the first failure has then already
gone through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2504_04704_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2504_04704_b200 import binding as b
    b.load_library()
    return b


def _case(seed, B, H, D, S_cap, seq, stat):
    K, V = synth.make_kv(B, H, S_cap, D, seed=seed, device="cuda:0")
    return (K, V, torch.tensor(seq, dtype=torch.int32, device="cuda:0"),
            torch.tensor(stat, dtype=torch.int32, device="cuda:0"))


def _run_both(binding, oracle, plan, ws, case, max_chunks, give_idx):
    """Same inputs through the workspace entry point, the no-allocation one and the oracle."""
    B, H, k = plan.cfg.B, plan.cfg.H_kv, plan.k
    K, V, seq, stat = case
    Ka, Va, seqa, stata = K.clone(), V.clone(), seq.clone(), stat.clone()
    Kb, Vb, seqb, statb = K.clone(), V.clone(), seq.clone(), stat.clone()
    idxa = torch.full((B, H, max_chunks * k), -1, dtype=torch.int32, device="cuda:0") if give_idx else None
    idxb = idxa.clone() if give_idx else None
    status = torch.full((4,), -7, dtype=torch.int32, device="cuda:0")       # caller-owned, made before the call
    plan.compress_append(Ka, Va, seqa, stata, ws, max_new_chunks=max_chunks, idx_out=idxa)
    want_status = plan.read_status(ws)
    plan.compress_append_noalloc(Kb, Vb, seqb, statb, max_new_chunks=max_chunks, idx_out=idxb, status_out=status)
    torch.cuda.synchronize()
    assert status.tolist()[:3] == want_status[:3]
    assert torch.equal(seqa, seqb) and torch.equal(stata, statb)
    assert torch.equal(Ka, Kb) and torch.equal(Va, Vb)
    if give_idx:
        assert torch.equal(idxa, idxb)
    assert not torch.equal(seqb, seq), "the case must trigger at least one compression"
    # the oracle's replay of the same append: lengths, rows up to the new length, kept positions
    Kr, Vr, seqr, statr, kept = oracle.compress_append(synth.to_bits(K), synth.to_bits(V), seq.cpu().numpy(),
                                                       stat.cpu().numpy(), plan.cfg.lag, k)
    assert seqb.tolist() == seqr.tolist() and statb.tolist() == statr.tolist()
    Kg, Vg = synth.to_bits(Kb), synth.to_bits(Vb)
    for b in range(B):
        m = int(seqr[b])
        np.testing.assert_array_equal(Kg[b, :, :m], Kr[b, :, :m])
        np.testing.assert_array_equal(Vg[b, :, :m], Vr[b, :, :m])
        if give_idx and kept[b].shape[1]:
            np.testing.assert_array_equal(idxb[b, :, :kept[b].shape[1]].cpu().numpy(), kept[b])
    return status.tolist()


def test_noalloc_matches_workspace_entry_point_twice_in_a_row(binding, oracle):
    B, H, D, sink, L, k = 3, 2, 128, 8, 64, 16
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace(3)
    # first call: kept positions parked in the library's scratch (no idx_out), several chunks
    c1 = _case(101, B, H, D, 600, [sink + 4 * L + 3, sink + 2 * L, sink + 2 * L - 1], [sink, sink, sink])
    st1 = _run_both(binding, oracle, plan, ws, c1, 3, give_idx=False)
    assert st1[0] == 0
    # second call right behind it, other data and lengths: nothing of the first call may leak in
    c2 = _case(202, B, H, D, 600, [sink + 3 * k + 2 * L + 9, sink + 3 * L + 1, sink + L], [sink + 3 * k, sink, sink])
    st2 = _run_both(binding, oracle, plan, ws, c2, 3, give_idx=True)
    assert st2[0] == 0
    # third: a device-side error code must show up in status_out and must not stick afterwards
    c3 = _case(303, B, H, D, 600, [sink + 5 * L, sink + 2 * L, sink + 2 * L], [sink, sink, sink])   # needs 4 chunks
    K, V, seq, stat = c3
    status = torch.zeros(4, dtype=torch.int32, device="cuda:0")
    plan.compress_append_noalloc(K, V, seq, stat, max_new_chunks=3, status_out=status)
    assert status.tolist()[0] == binding.LAGKV_ECAPACITY
    # without status_out the code waits in the built-in scratch until it is read (or the next call clears it)
    plan.compress_append_noalloc(K, V, seq, stat, max_new_chunks=3)
    assert plan.read_status(None)[0] == binding.LAGKV_ECAPACITY
    assert plan.read_status(None)[0] == 0
    st4 = _run_both(binding, oracle, plan, ws, c1, 3, give_idx=False)
    assert st4[0] == 0


def test_noalloc_refuses_what_does_not_fit(binding):
    """256 + B*H*max_new_chunks*k*4 bytes beyond the built-in array: refused, nothing touched."""
    B, H, D, sink, L, k = 64, 8, 128, 4, 512, 512
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    assert plan.workspace_bytes(2) > binding.NOALLOC_SCRATCH_BYTES
    K = torch.zeros((B, H, 8, D), dtype=torch.bfloat16, device="cuda:0")
    V = torch.zeros_like(K)
    seq = torch.full((B,), 8, dtype=torch.int32, device="cuda:0")
    stat = torch.full((B,), 4, dtype=torch.int32, device="cuda:0")
    with pytest.raises(binding.LagKVError) as e:
        plan.compress_append_noalloc(K, V, seq, stat, max_new_chunks=2)
    assert e.value.code == binding.LAGKV_ENOALLOC_LIMIT
    # an argument the host refuses must not clear what the previous call left in the scratch
    small = binding.Plan(2, 1, D, 4, 8, keep_k=8, device=0)
    k2, v2 = torch.zeros((2, 1, 64, D), dtype=torch.bfloat16, device="cuda:0"), torch.zeros((2, 1, 64, D), dtype=torch.bfloat16, device="cuda:0")
    s2 = torch.tensor([4 + 5 * 8, 4], dtype=torch.int32, device="cuda:0")
    t2 = torch.tensor([4, 4], dtype=torch.int32, device="cuda:0")
    small.compress_append_noalloc(k2, v2, s2, t2, max_new_chunks=1)             # needs 4 chunks: ECAPACITY on the device
    with pytest.raises(binding.LagKVError) as e2:
        small.compress_append_noalloc(k2, k2, s2, t2, max_new_chunks=1)         # K and V alias: refused on the host
    assert e2.value.code == binding.LAGKV_EINVAL
    assert small.read_status(None)[0] == binding.LAGKV_ECAPACITY
    assert "scratch" in binding.status_string(binding.LAGKV_ENOALLOC_LIMIT)
    assert seq.tolist() == [8] * B
    # with idx_out supplied only the status block is needed, so the same shape is accepted
    idx = torch.full((B, H, 2 * k), -1, dtype=torch.int32, device="cuda:0")
    plan.compress_append_noalloc(K, V, seq, stat, max_new_chunks=2, idx_out=idx)
    torch.cuda.synchronize()
    assert seq.tolist() == [8] * B          # rest < 2L: skipped on the device
