"""qasr_tcs_block_noalloc -- the entry point for callers that may not allocate device memory
(fixed-budget streaming callbacks, serving plugins whose enqueue hook must stay off the allocator,
processes whose device memory is already reserved).  It must give exactly what qasr_tcs_block and
the CPU oracle give, call after call, although every call reuses the same static scratch array, it
must refuse problems that do not fit that array, and an error that an asynchronous call leaves in
the shared status word must reach the next waiting caller exactly once.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu


def _block(seed, B, Ci, Co, T, K, stride, dil):
    rng = workloads.rng_for(seed)
    x = workloads.draw_input(rng, B, Ci, T)
    bld = workloads._Builder(rng, "live", True, False)
    bld.conv("tcs", "blk", 0, Ci, Co, K, stride, dil, True, workloads.MS_INPUT)
    return x, bld.layers[0]


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_noalloc_matches_tcs_block_on_two_calls_in_a_row():
    import paper_2103_16827_b200 as q
    ctx = q.Context(0)
    cases = [(11, 4, 256, 256, 800, 33, 1, 1), (12, 2, 512, 256, 640, 75, 1, 1), (13, 2, 64, 128, 1000, 33, 2, 1)]
    outs = []
    n_calls = 0
    for seed, B, Ci, Co, T, K, stride, dil in cases:
        x, L = _block(seed, B, Ci, Co, T, K, stride, dil)
        args = (_dev(x), _dev(L["w_dw"]), stride, dil, _dev(L["m_dw"]), _dev(L["s_dw"]), _dev(L["w"]),
                _dev(L["bias"]), L["max_abs_bias"], _dev(L["m"]), _dev(L["s"]), True)
        want = ctx.tcs_block(*args)
        ctx.poll_status()
        ref = oracle.run_layer(L, {0: x})["y"]
        assert np.array_equal(want.cpu().numpy(), ref), "qasr_tcs_block differs from the oracle (case %d)" % seed
        y = torch.empty_like(want)
        torch.cuda.synchronize()
        # device memory in use must not move across the call itself (the kernels it runs were already
        # loaded by the qasr_tcs_block call above, so nothing legitimate is left to allocate)
        free_before = torch.cuda.mem_get_info()[0]
        got = q.tcs_block_noalloc(*args, y=y, device=0, wait=True)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if n_calls > 0:
            assert free_after == free_before, "the call changed the amount of free device memory"
        n_calls += 1
        assert torch.equal(got, want), "no-alloc result differs from qasr_tcs_block (case %d)" % seed
        assert np.array_equal(got.cpu().numpy(), ref), "no-alloc result differs from the oracle (case %d)" % seed
        assert int((want != 0).sum()) > want.numel() // 4
        outs.append(got.clone())
    # the same first problem again: stale scratch contents from the other shapes must not leak in
    seed, B, Ci, Co, T, K, stride, dil = cases[0]
    x, L = _block(seed, B, Ci, Co, T, K, stride, dil)
    y = torch.empty_like(outs[0])
    q.tcs_block_noalloc(_dev(x), _dev(L["w_dw"]), stride, dil, _dev(L["m_dw"]), _dev(L["s_dw"]), _dev(L["w"]),
                        _dev(L["bias"]), L["max_abs_bias"], _dev(L["m"]), _dev(L["s"]), True, y=y, wait=True)
    assert torch.equal(y, outs[0])
    assert np.array_equal(y.cpu().numpy(), oracle.run_layer(L, {0: x})["y"])
    ctx.close()


def test_noalloc_status_word_is_shared_and_sticky():
    """An out-of-range shift seen by an asynchronous call (wait = 0) is not lost: the next call that waits
    reports QASR_ERR_RANGE once and clears it, the call after that succeeds."""
    import paper_2103_16827_b200 as q
    x, L = _block(21, 8, 64, 64, 256, 33, 1, 1)
    bad_shift = L["s_dw"].copy()
    bad_shift[3] = 63
    common = (_dev(L["w"]), _dev(L["bias"]), L["max_abs_bias"], _dev(L["m"]), _dev(L["s"]), True)
    y = torch.empty((8, 64, 256), dtype=torch.int8, device="cuda")
    xd, wd, md = _dev(x), _dev(L["w_dw"]), _dev(L["m_dw"])
    q.tcs_block_noalloc(xd, wd, 1, 1, md, _dev(bad_shift), *common, y=y, wait=False)     # returns 0: nothing read back yet
    with pytest.raises(q.QasrError) as e:
        q.tcs_block_noalloc(xd, wd, 1, 1, md, _dev(L["s_dw"]), *common, y=y, wait=True)
    assert e.value.code == -4
    q.tcs_block_noalloc(xd, wd, 1, 1, md, _dev(L["s_dw"]), *common, y=y, wait=True)      # cleared
    assert np.array_equal(y.cpu().numpy(), oracle.run_layer(L, {0: x})["y"])


def test_noalloc_rejects_what_does_not_fit_or_is_malformed():
    import paper_2103_16827_b200 as q
    B, Ci, Co, T = 40, 512, 64, 1024                    # depthwise output 20 MiB > 16 MiB
    assert B * Ci * T > q.NOALLOC_SCRATCH_BYTES
    x = torch.zeros((B, Ci, T), dtype=torch.int8, device="cuda")
    wd = torch.zeros((Ci, 33), dtype=torch.int8, device="cuda")
    wp = torch.zeros((Co, Ci), dtype=torch.int8, device="cuda")
    m = torch.ones(Ci, dtype=torch.int32, device="cuda")
    s = torch.ones(Ci, dtype=torch.uint8, device="cuda")
    y = torch.zeros((B, Co, T), dtype=torch.int8, device="cuda")
    with pytest.raises(q.QasrError) as e:
        q.tcs_block_noalloc(x, wd, 1, 1, m, s, wp, None, 0, m[:Co], s[:Co], True, y=y)
    assert e.value.code == -11 and "static scratch" in str(e.value)
    with pytest.raises(q.QasrError) as e:
        q.tcs_block_noalloc(x[:1], wd[:, :32].contiguous(), 1, 1, m, s, wp, None, 0, m[:Co], s[:Co], True, y=y[:1])
    assert e.value.code == -2
    with pytest.raises(q.QasrError) as e:
        q.tcs_block_noalloc(x[:1], wd, 1, 1, m, s, wp, None, 0, m[:Co], s[:Co], True, y=x[:1])
    assert e.value.code == -10
