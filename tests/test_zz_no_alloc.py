"""moe_permute_static -- the entry point for callers that may not allocate device memory (a
plug-in inside an engine that owns all GPU memory, a loop that cannot afford cudaMalloc's
device-wide synchronisation).  Its scratch is a fixed array inside the library, so the test is
simple: called through the C ABI it must give exactly what moe_permute gives with a caller
workspace, on two calls in a row (the second, smaller problem runs over whatever the first left
in the shared array), and it must refuse shapes beyond the array's size.

Collected last on purpose: a run that stops at the first failure has then already run every other
test."""
import numpy as np
import pytest
import torch

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import binding as B
from paper_2604_08133_b200 import synth

pytestmark = pytest.mark.gpu


def _routing(T, N, K, kb, budget, seed):
    g = torch.Generator().manual_seed(seed)
    p = orc.softmax_scores(torch.randn(T, N, generator=g, dtype=torch.float64).numpy())
    idx, sc = orc.topk_sorted(p, K)
    n_sel = orc.n_sel_from_mask(orc.alloc_t_select_threshold(sc, kb, budget))
    return torch.from_numpy(idx).cuda(), torch.from_numpy(sc).cuda(), torch.from_numpy(n_sel).cuda()


def _outputs(T, N, K, H, budget):
    return dict(off=torch.full((N + 1,), -3, dtype=torch.int32, device="cuda"),
                tok=torch.full((budget,), -3, dtype=torch.int32, device="cuda"),
                wgt=torch.full((budget,), -3.0, dtype=torch.float32, device="cuda"),
                pos=torch.full((T, K), -3, dtype=torch.int32, device="cuda"),
                xp=torch.full((budget, H), -3.0, dtype=torch.bfloat16, device="cuda"))


def _one_case(T, N, K, kb, mult, seed):
    H = 128
    budget = int(mult * T)
    idx, sc, n_sel = _routing(T, N, K, kb, budget, seed)
    x = synth.normal_bf16((T, H), 1.0, synth.stream_key(9, seed)).cuda()
    shape = B.make_shape(T, H, N, 64, 0, K, kb)
    ref, got = _outputs(T, N, K, H, budget), _outputs(T, N, K, H, budget)
    st_ref = torch.zeros(1, dtype=torch.int32, device="cuda")
    st_got = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = B.new_workspace(shape, budget)
    B.moe_permute(shape, x, idx, sc, n_sel, budget, ref["off"], ref["tok"], ref["wgt"], ref["pos"], ref["xp"],
                  st_ref, ws)
    B.moe_permute_static(shape, x, idx, sc, n_sel, budget, got["off"], got["tok"], got["wgt"], got["pos"],
                         got["xp"], st_got)
    torch.cuda.synchronize()
    assert st_ref.item() == 0 and st_got.item() == 0
    for k in ref:                                   # integer and byte outputs: bit-exact
        assert torch.equal(ref[k].view(torch.int16) if ref[k].dtype == torch.bfloat16 else ref[k],
                           got[k].view(torch.int16) if got[k].dtype == torch.bfloat16 else got[k]), k
    assert int(got["off"][-1]) == budget
    # and directly against the oracle's permutation of the same routing
    want = orc.permute(idx.cpu().numpy(), sc.cpu().numpy(), n_sel.cpu().numpy(), N)
    assert np.array_equal(got["off"].cpu().numpy(), want["expert_offsets"])
    assert np.array_equal(got["tok"].cpu().numpy(), want["perm_token"])
    assert np.array_equal(got["wgt"].cpu().numpy(), want["perm_weight"])
    assert np.array_equal(got["pos"].cpu().numpy(), want["pair_pos"])
    assert torch.equal(got["xp"].cpu(), x.cpu()[torch.from_numpy(want["perm_token"]).long()])


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    _one_case(T=4096, N=64, K=6, kb=1, mult=4.5, seed=1)     # 8192 counters
    _one_case(T=777, N=16, K=4, kb=0, mult=1.3, seed=2)      # a smaller problem over the stale array
    _one_case(T=4096, N=64, K=6, kb=1, mult=2.0, seed=3)


def test_static_scratch_at_exactly_its_size():
    _one_case(T=32768, N=64, K=2, kb=1, mult=1.5, seed=4)    # 64 * 1024 = 65536 counters: the whole array
    _one_case(T=32737, N=64, K=2, kb=0, mult=0.7, seed=5)    # the last segment holds one token


def test_static_scratch_rejects_shapes_beyond_its_size():
    shape = B.make_shape(32800, 128, 64, 64, 0, 2, 1)         # 64 * 1025 = 65600 counters: just past the array
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MoeError) as ei:
        B.moe_permute_static(shape, None, dummy, dummy.float(), dummy, 32800, dummy, dummy, dummy.float(), dummy, None,
                             dummy)
    assert ei.value.status == B.MOE_ERR_WORKSPACE
    bad = B.make_shape(64, 128, 8, 100, 0, 2, 1)              # I not a multiple of 64: refused like moe_permute does
    with pytest.raises(B.MoeError) as ei:
        B.moe_permute_static(bad, None, dummy, dummy.float(), dummy, 64, dummy, dummy, dummy.float(), dummy, None, dummy)
    assert ei.value.status == B.MOE_ERR_ARG

    T, N, K = 40000, 64, 2                                    # 64 * 1250 = 80000 counters > 65536
    shape = B.make_shape(T, 128, N, 64, 0, K, 1)
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MoeError) as ei:
        B.moe_permute_static(shape, None, dummy, dummy.float(), dummy, T, dummy, dummy, dummy.float(), dummy, None,
                             dummy)
    assert ei.value.status == B.MOE_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert int(dummy.sum()) == 0                              # nothing was launched
