"""The workspace-free router/selection entry point against the regular one.

qtale_router_select_static exists for callers that are not allowed to allocate
device memory (a plugin living inside someone else's memory pool, a loop that
bans allocator calls after start-up).  It keeps its scratch inside the library
image, shared by all calls, so the checks here are: same outputs as
qtale_router_select, bit for bit, on two different calls in a row (the second
one must not be disturbed by what the first left in the shared scratch), and a
clean refusal instead of a launch when the arguments are bad or the call has
more tokens than the built-in scratch was sized for; the call must also leave
the amount of device memory in use exactly as it found it.

Collected last on purpose: if this file fails, every other test has already run.
"""
import numpy as np
import pytest

from paper_2602_10431_b200 import inputs

pytestmark = pytest.mark.gpu


def _outputs(torch, dev, T, B):
    return dict(scores=torch.zeros(T, dtype=torch.float32, device=dev),
                idx=torch.full((T,), -1, dtype=torch.int32, device=dev),
                n_exec=torch.zeros(1, dtype=torch.int32, device=dev),
                cu_exec=torch.zeros(B + 1, dtype=torch.int32, device=dev),
                pos=torch.full((T,), -1, dtype=torch.int32, device=dev))


def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row():
    import torch
    from paper_2602_10431_b200 import api
    api.lib()
    dev = torch.device("cuda", 0)
    calls = [
        # (T, d, cu_seqlens, mode, theta, k)
        (1000, 512, [0, 100, 100, 650, 1000], api.SELECT_THRESHOLD, 0.5, 0),
        (4096, 1024, [0, 2048, 4096], api.SELECT_TOPK, 0.0, 1357),
    ]
    for T, d, cu, mode, theta, k in calls:
        x = api.to_device_bf16(inputs.hidden_states(T, T, d), dev)
        w = torch.from_numpy(inputs.round_bf16((inputs.normal(T, 5, d) * 0.02).astype(np.float32))).to(dev)
        cud = torch.tensor(cu, dtype=torch.int32, device=dev)
        want = api.router_select(x, w, 0.05, cud, mode, theta=theta, k=k)
        outs = _outputs(torch, dev, T, len(cu) - 1)
        torch.cuda.synchronize()
        held, free1 = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        got = api.router_select_static(x, w, 0.05, cud, mode, outs, theta=theta, k=k)
        torch.cuda.synchronize()
        # the call took no device memory, neither from torch's pool nor from the driver (either
        # figure may shrink meanwhile: Python frees earlier temporaries when it pleases)
        assert torch.cuda.memory_allocated() <= held and torch.cuda.mem_get_info()[0] >= free1
        assert api.device_status() == 0
        n = int(want["n_exec"].item())
        assert int(got["n_exec"].item()) == n and n > 0
        # integer outputs and the fp32 scores are the same kernel's: identical bits
        for key in ("scores", "idx", "cu_exec", "pos"):
            assert torch.equal(got[key], want[key]), key


def test_static_scratch_entry_point_refuses_bad_arguments():
    import torch
    from paper_2602_10431_b200 import api
    L = api.lib()
    args = [None, 4, 64, None, 0.0, None, None, None, 1, None, 0, 0.5, 0, None, None, None, None, None, None]
    assert L.qtale_router_select_static(*args) == -1      # null pointers: nothing launched
    # more tokens than the built-in scratch is sized for: refused, nothing launched or written
    dev = torch.device("cuda", 0)
    T = api.ROUTER_STATIC_MAX_TOKENS + 1
    sc = torch.rand(T, device=dev)
    cud = torch.tensor([0, T], dtype=torch.int32, device=dev)
    outs = _outputs(torch, dev, T, 1)
    with pytest.raises(api.QtaleError, match="capacity"):
        api.router_select_static(None, None, 0.0, cud, api.SELECT_THRESHOLD, outs, scores_override=sc)
    torch.cuda.synchronize()
    assert int(outs["n_exec"].item()) == 0 and bool((outs["idx"] == -1).all())
    # the largest accepted call still works
    T = api.ROUTER_STATIC_MAX_TOKENS
    outs = _outputs(torch, dev, T, 1)
    cud = torch.tensor([0, T], dtype=torch.int32, device=dev)
    api.router_select_static(None, None, 0.0, cud, api.SELECT_TOPK, outs, k=T // 3, scores_override=sc[:T])
    want = api.router_select(None, None, 0.0, cud, api.SELECT_TOPK, k=T // 3, scores_override=sc[:T])
    assert int(outs["n_exec"].item()) == T // 3 and torch.equal(outs["idx"], want["idx"])
