"""GPU parity of the individual entry points against the CPU oracle.

Every call goes through the C ABI (paper_2602_10431_b200.api is marshalling
only).  Integer / index results must be bit-exact; floating point within the
tolerances written next to each check."""
import numpy as np
import pytest

import oracle
from paper_2602_10431_b200 import inputs
from tests.gpu_util import act_eps, assert_selection_matches, rel_fro, round_act

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2602_10431_b200 import api
    api.lib()
    return api, torch, torch.device("cuda", 0)


def _check_select(api, torch, r, p_ref, m_ref, cu, pos0=None, threshold=None):
    idx_ref, n_ref, cue_ref, pos_ref = oracle.compact_indices(m_ref, cu)
    n = int(r["n_exec"].item())
    idx = r["idx"].cpu().numpy()
    assert_selection_matches(idx, n, p_ref, m_ref, threshold)
    if n == n_ref:
        assert np.array_equal(idx[:n], idx_ref)
        assert np.array_equal(r["cu_exec"].cpu().numpy(), cue_ref)
        seq = np.searchsorted(cu, idx_ref, side="right") - 1
        want_pos = pos_ref + (0 if pos0 is None else pos0[seq])
        assert np.array_equal(r["pos"].cpu().numpy()[:n], want_pos)
    assert (idx[n:] == -1).all()  # entries past the count are untouched
    assert api.device_status() == 0


@pytest.mark.parametrize("T,d,cu", [
    (256, 256, [0, 128, 256]),
    (1000, 512, [0, 100, 100, 650, 1000]),      # empty sequence, ragged
    (37, 4096, [0, 37]),                         # fewer rows than one warp group
    (5000, 1024, [0, 1, 2, 3, 4999, 5000]),
])
def test_router_select_threshold_and_topk(env, T, d, cu):
    api, torch, dev = env
    cu = np.array(cu, np.int32)
    x = inputs.hidden_states(T, T, d)
    w = inputs.round_bf16((inputs.normal(T, 5, d) * 0.02).astype(np.float32))
    p_ref, z = oracle.router_scores(x, w, 0.05, return_logits=True)
    xd, wd, cud = api.to_device_bf16(x, dev), torch.from_numpy(w).to(dev), torch.from_numpy(cu).to(dev)
    for theta in [0.5, 0.3, 0.0, 1.5]:
        r = api.router_select(xd, wd, 0.05, cud, api.SELECT_THRESHOLD, theta=theta)
        # scores: fp64 accumulation on both sides; equal to the last fp32 bit in practice
        assert np.abs(r["scores"].cpu().numpy() - p_ref).max() <= 1e-7
        _check_select(api, torch, r, p_ref, oracle.select_threshold(p_ref, theta), cu, threshold=theta)
    for ratio in [0.0, 0.5, 0.9, 1.0]:
        k = api.topk_count(ratio, T)
        r = api.router_select(xd, wd, 0.05, cud, api.SELECT_TOPK, k=k)
        m = oracle.select_topk(p_ref, k)
        assert int(r["n_exec"].item()) == k
        _check_select(api, torch, r, p_ref, m, cu)


def test_router_select_padding_override_ties_pos0(env):
    api, torch, dev = env
    T = 777
    cu = np.array([0, 300, 777], np.int32)
    pos0 = np.array([5, 2048], np.int32)
    p = inputs.beta22(3, 1, T).astype(np.float32)
    p[100:140] = p[50]                 # a run of equal scores for the tie rule
    valid = (inputs.uniform(3, 2, T) > 0.25).astype(np.uint8)
    pd, vd = torch.from_numpy(p).to(dev), torch.from_numpy(valid).to(dev)
    cud, p0d = torch.from_numpy(cu).to(dev), torch.from_numpy(pos0).to(dev)
    r = api.router_select(None, None, 0.0, cud, api.SELECT_THRESHOLD, theta=float(p[50]),
                          scores_override=pd, valid=vd, pos0=p0d)
    assert np.array_equal(r["scores"].cpu().numpy(), p)
    _check_select(api, torch, r, p, oracle.select_threshold(p, float(p[50]), valid), cu, pos0)
    n_valid = int(valid.sum())
    for k in [1, 17, int((p[valid == 1] > p[50]).sum()) + 7, n_valid]:
        r = api.router_select(None, None, 0.0, cud, api.SELECT_TOPK, k=k, scores_override=pd,
                              valid=vd, pos0=p0d)
        _check_select(api, torch, r, p, oracle.select_topk(p, k, valid), cu, pos0)


def _select_case(api, torch, dev, p, cu, mode, k=0, theta=0.5, valid=None):
    pd = torch.from_numpy(p).to(dev)
    vd = None if valid is None else torch.from_numpy(valid).to(dev)
    r = api.router_select(None, None, 0.0, torch.from_numpy(cu).to(dev), mode, theta=theta, k=k,
                          scores_override=pd, valid=vd)
    m = oracle.select_topk(p, k, valid) if mode == api.SELECT_TOPK else oracle.select_threshold(p, theta, valid)
    _check_select(api, torch, r, p, m, cu, threshold=None if mode == api.SELECT_TOPK else theta)
    return int(r["n_exec"].item())


def test_topk_selection_with_many_equal_scores(env):
    """Equal scores are ordered by token index.  All scores equal, or a block of more equal
    scores than the in-kernel candidate buffer holds (1024), takes the radix-select path of
    the cut-off; a few equal scores take the ranking path; both across several CTAs."""
    api, torch, dev = env
    T = 5000
    cu = np.array([0, 1200, 1200, 3100, 5000], np.int32)
    same = np.full(T, 0.625, np.float32)
    for k in [1, 1234, 4999, 5000]:
        assert _select_case(api, torch, dev, same, cu, api.SELECT_TOPK, k=k) == k
    p = inputs.beta22(41, 1, T).astype(np.float32)
    p[700:2900] = p[10]                                         # 2200 equal scores in the middle
    valid = (inputs.uniform(41, 2, T) > 0.1).astype(np.uint8)
    above = int(((p > p[10]) & (valid == 1)).sum())
    for k in [above, above + 1, above + 1500, above + int(((p == p[10]) & (valid == 1)).sum()), above + 2300]:
        _select_case(api, torch, dev, p, cu, api.SELECT_TOPK, k=k, valid=valid)
    p = inputs.beta22(41, 3, T).astype(np.float32)
    p[::7] = p[3]                                               # 715 equal scores, interleaved
    for k in [int((p > p[3]).sum()) + 100, 2500]:
        _select_case(api, torch, dev, p, cu, api.SELECT_TOPK, k=k)
    # scores outside [0, 1) fall into the end bins of the histogram and are still ordered exactly
    p = (inputs.normal(41, 4, T) * 2).astype(np.float32)
    for k in [17, 2500, 4000]:
        _select_case(api, torch, dev, p, cu, api.SELECT_TOPK, k=k)


@pytest.mark.parametrize("T,B", [(65536, 16), (200000, 5), (1300000, 3)])
def test_selection_at_scale(env, T, B):
    """65536 tokens in 16 sequences with Beta(2,2) scores is the 13B-shaped stack's selection
    (threshold from the closed-form quantile and top-k at ratio 0.7); the larger cases give a CTA
    more tokens than threads, and more than it keeps in shared memory."""
    api, torch, dev = env
    p = inputs.beta22(43, 1, T).astype(np.float32)
    cu = (np.arange(B + 1, dtype=np.int64) * T // B).astype(np.int32)
    n = _select_case(api, torch, dev, p, cu, api.SELECT_THRESHOLD, theta=0.3)
    assert abs(n / T - (1 - (3 * 0.3 ** 2 - 2 * 0.3 ** 3))) < 0.01   # Beta(2,2) tail above 0.3
    k = api.topk_count(0.7, T) if T == 65536 else 500
    assert _select_case(api, torch, dev, p, cu, api.SELECT_TOPK, k=k) == k


@pytest.mark.parametrize("T,d,h", [(100, 256, 8), (777, 1000, 5), (2100, 4096, 64), (33, 64, 17)])
def test_router_mlp_scores(env, T, d, h):
    """MLP router (Eq. 2) against the oracle's fp64 evaluation: the hidden layer runs on the
    tensor cores with fp64 accumulation across 64-feature chunks, so the probabilities agree to
    1e-6 and a threshold decision on them is the oracle's outside the 1e-6 band.  Covers a
    feature count that is not a multiple of the chunk, hidden widths that are not multiples of 8
    and a partial last row block."""
    api, torch, dev = env
    x = inputs.hidden_states(80 + h, T, d)
    w1 = inputs.round_bf16((inputs.normal(81, 1, h * d) * 0.05).astype(np.float32)).reshape(h, d)
    b1 = (inputs.normal(81, 2, h) * 0.5).astype(np.float32)
    w2 = (inputs.normal(81, 3, 2 * h) * 0.5).astype(np.float32).reshape(2, h)
    b2 = np.array([0.2, -0.1], np.float32)
    p_ref = oracle.router_mlp_scores(x, w1, b1, w2, b2)
    sc = api.router_mlp_scores(api.to_device_bf16(x, dev), api.to_device_bf16(w1, dev),
                               torch.from_numpy(b1).to(dev), torch.from_numpy(w2).to(dev), b2)
    got = sc.cpu().numpy()
    assert api.device_status() == 0
    assert np.abs(got - p_ref).max() <= 1e-6
    assert 0.05 < p_ref.mean() < 0.95
    cu = np.array([0, T // 3, T], np.int32)
    theta = float(np.median(p_ref))
    r = api.router_select(None, None, 0.0, torch.from_numpy(cu).to(dev), api.SELECT_THRESHOLD, theta=theta,
                          scores_override=sc)
    _check_select(api, torch, r, p_ref, oracle.select_threshold(p_ref, theta), cu, threshold=theta)


@pytest.mark.parametrize("n", [1, 777, 262144, 1500000])
def test_theta_for_ratio_matches_the_sorted_quantile(env, n):
    """The device-side quantile is a selection, so theta and the count must equal the oracle's
    sort-based ones bit for bit: padding, ties at the cut, ratios 0 and 1, 32 layers x 8192
    pooled scores (the model-prefill calibration size) and a case of many CTAs."""
    api, torch, dev = env
    p = inputs.beta22(61, 1, n).astype(np.float32)
    if n > 700:
        p[100:700] = p[3]
    valid = (inputs.uniform(61, 2, n) > 0.15).astype(np.uint8)
    pd, vd = torch.from_numpy(p).to(dev), torch.from_numpy(valid).to(dev)
    for ratio in [0.0, 0.3, 0.75, 1.0]:
        for v_np, v_d in [(None, None), (valid, vd)]:
            if v_np is not None and v_np.sum() == 0:
                continue
            th_ref, c_ref = oracle.theta_for_ratio(p, ratio, v_np)
            th, c = api.theta_for_ratio(pd, ratio, valid=v_d)
            assert api.device_status() == 0
            assert float(th.item()) == np.float32(th_ref) and int(c.item()) == c_ref
    # Eq. 9 with that theta executes the requested share
    th, c = api.theta_for_ratio(pd, 0.5)
    r = api.router_select(None, None, 0.0, torch.tensor([0, n], dtype=torch.int32, device=dev),
                          api.SELECT_THRESHOLD, theta=float(th.item()), scores_override=pd)
    assert int(r["n_exec"].item()) == int(c.item()) >= api.topk_count(0.5, n)


def test_inconsistent_cu_seqlens_is_reported_not_followed(env):
    """cu_seqlens lives on the device, so the kernel checks it: offsets that do not end at T
    (or are not ascending) give QTALE_ERR_SHAPE in the status word, tokens outside
    [cu[0], cu[B]) never execute, and nothing outside the B + 1 entries is read."""
    api, torch, dev = env
    T, d = 256, 256
    x = inputs.hidden_states(31, T, d)
    w = inputs.round_bf16((inputs.normal(31, 5, d) * 0.02).astype(np.float32))
    xd, wd = api.to_device_bf16(x, dev), torch.from_numpy(w).to(dev)
    p_ref = oracle.router_scores(x, w, 0.0)
    for cu, lo, hi in [([0, 100, 200], 0, 200), ([10, 100, 256], 10, 256), ([0, 200, 100, 256], 0, 256)]:
        cud = torch.tensor(cu, dtype=torch.int32, device=dev)
        r = api.router_select(xd, wd, 0.0, cud, api.SELECT_THRESHOLD, theta=0.0)   # everything executes
        torch.cuda.synchronize()
        assert api.device_status() == -3                        # QTALE_ERR_SHAPE
        n = int(r["n_exec"].item())
        idx = r["idx"].cpu().numpy()
        assert n == hi - lo and np.array_equal(idx[:n], np.arange(lo, hi)) and (idx[n:] == -1).all()
        assert np.abs(r["scores"].cpu().numpy() - p_ref).max() <= 1e-7
    # a consistent list right afterwards: clean status
    r = api.router_select(xd, wd, 0.0, torch.tensor([0, 0, 256], dtype=torch.int32, device=dev),
                          api.SELECT_TOPK, k=17)
    assert api.device_status() == 0 and int(r["n_exec"].item()) == 17


def test_index_bookkeeping(env):
    api, torch, dev = env
    T = 500
    cu = np.array([0, 200, 200, 500], np.int32)
    mask = (inputs.uniform(4, 1, T) > 0.6).astype(np.uint8)
    idx, n, cue, pos = oracle.compact_indices(mask, cu)
    r = api.index_bookkeeping(torch.from_numpy(idx).to(dev), n, T, torch.from_numpy(cu).to(dev))
    assert int(r["n_exec"].item()) == n
    assert np.array_equal(r["cu_exec"].cpu().numpy(), cue)
    assert np.array_equal(r["pos"].cpu().numpy()[:n], pos)
    r = api.index_bookkeeping(None, 0, T, torch.from_numpy(cu).to(dev))
    assert int(r["n_exec"].item()) == 0 and not r["cu_exec"].cpu().numpy().any()


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("T,d,ratio", [(256, 256, 0.5), (300, 4096, 0.7), (64, 5120, 1.0), (129, 512, 0.0)])
def test_compact_and_scatter(env, T, d, ratio, act):
    api, torch, dev = env
    x = inputs.hidden_states(T + d, T, d)
    mask = (inputs.uniform(T, 3, T) < ratio).astype(np.uint8)
    idx, n, _, _ = oracle.compact_indices(mask, np.array([0, T], np.int32))
    idx_d = torch.full((T,), 0, dtype=torch.int32, device=dev)
    idx_d[:n] = torch.from_numpy(idx).to(dev)
    n_d = torch.tensor([n], dtype=torch.int32, device=dev)
    gam = (1 + 0.1 * inputs.normal(T, 7, d)).astype(np.float32)
    xd = api.to_device_bf16(x, dev)
    xc, hn = api.compact(xd, idx_d, n_d, torch.from_numpy(gam).to(dev), 1e-5, act_dtype=act)
    xc_h, hn_h = api.to_host_f32(xc), api.to_host_f32(hn)
    assert np.array_equal(xc_h[:n], oracle.gather_rows(x, idx))       # byte copy
    assert not xc_h[n:].any() and not hn_h[n:].any()                  # rows past the count untouched
    if n:
        ref = oracle.rmsnorm(x[idx], gam, 1e-5)
        # fp32 arithmetic, one rounding to the activation format: half an ulp relative, plus slack
        assert np.all(np.abs(hn_h[:n] - ref) <= np.abs(ref) * 2 * act_eps(act) + 1e-6)
    f = inputs.gaussian_f32(T, 9, T, d, 0.5)
    x2 = api.scatter_add(xd.clone(), xc, torch.from_numpy(f).to(dev), idx_d, n_d)
    out = api.to_host_f32(x2)
    want = oracle.scatter_add(x, x[idx], f[:n], idx)
    assert np.array_equal(out[mask == 0], x[mask == 0])               # bypass rows bit-identical
    if n:
        assert np.array_equal(out[idx], inputs.round_bf16(want[idx]))  # one bf16 rounding of the fp32 sum


GEMM_CASES = [
    # M_cap, N, K, bits, group, m_dev
    (64, 128, 64, 4, 64, None),
    (256, 768, 256, 4, 64, None),          # config-1 QKV
    (256, 256, 688, 4, 64, 201),           # K not a multiple of the group (config-1 down projection)
    (300, 1376, 256, 4, 64, 211),          # N not a multiple of 128, ragged M
    (100, 256, 512, 4, 128, None),         # 128-token tiles
    (64, 384, 256, 3, 64, 1),              # 3-bit, a single token
    (520, 256, 1024, 3, 128, 513),         # 3-bit, several token tiles and a tail of one
    (256, 512, 128, 4, 128, 0),            # nothing to do
    (129, 384, 192, 4, 64, None),          # smallest CTA-pair case: three row tiles (one padded), one and a half K steps
    (700, 640, 384, 3, 128, 651),          # CTA-pair, 3-bit, five row tiles, ragged tokens over three tiles
    (64, 9600, 128, 4, 128, 37),           # decode kernel, half a row tile per CTA
    (48, 38016, 64, 3, 64, None),          # decode kernel, a whole row tile per CTA, 3-bit
    (33, 256, 704, 4, 64, 33),             # decode kernel, a quarter tile per CTA, four K groups, odd K blocks
    (64, 512, 4096, 3, 128, 58),           # decode kernel at the 7B-shaped K: 64 K blocks through the ring
    (64, 256, 11008, 4, 64, 38),           # decode kernel, K of the down projection: 172 K blocks
    (57, 384, 11008, 3, 128, None),        # the same in 3-bit, token count not a multiple of 8
    (200, 384, 320, 2, 64, 131),           # 2-bit (mixed 2&4-bit layers), single-CTA kernel, ragged tokens
    (700, 640, 384, 2, 128, 651),          # 2-bit, CTA-pair kernel
    (64, 9600, 192, 2, 64, 37),            # 2-bit, decode kernel (and split over K with a workspace)
    (40, 256, 4096, 2, 128, None),         # 2-bit, decode kernel, 64 K blocks
]


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("M,N,K,bits,group,m_dev", GEMM_CASES)
def test_wq_gemm_against_oracle(env, M, N, K, bits, group, m_dev, act):
    api, torch, dev = env
    a = inputs.activations(M + N, 11, M, K)
    wq = inputs.quantized_weight(K + bits, 12, N, K, bits, group)
    w_hat = oracle.dequantize_weight(wq)
    mm = M if m_dev is None else m_dev
    qw = api.QuantWeight(wq, dev)
    md = None if m_dev is None else torch.tensor([m_dev], dtype=torch.int32, device=dev)
    ad = api.to_device_act(a, act, dev)                       # N(0,1) bf16 values are exact in fp16 too
    y = api.wq_gemm(ad, qw, md, api.EPI_STORE_F32).cpu().numpy()
    assert api.device_status() == 0
    assert not y[mm:].any()                                   # rows past the count untouched
    if mm == 0:
        return
    ref = oracle.linear(a[:mm], w_hat)
    # kernel rounds the dequantised weight once to the 16-bit format (half an ulp relative per weight)
    assert rel_fro(y[:mm], ref) <= 6 * act_eps(act)
    # with the same rounding applied to the oracle's weights only fp32 summation order differs
    ref_b = oracle.linear(a[:mm], round_act(w_hat, act))
    assert np.abs(y[:mm] - ref_b).max() <= 1e-4 * max(1.0, np.abs(ref_b).max())
    yb = api.to_host_f32(api.wq_gemm(ad, qw, md, api.EPI_STORE_16))
    assert np.array_equal(yb[:mm], round_act(y[:mm], act))
    if M <= 64:
        # with a workspace the same product runs with the input dimension split over the SMs
        # (partial sums added in a fixed order): same tolerance, and bit-identical on a second run
        ws = torch.full((api.wq_gemm_workspace_bytes(),), 0xFF, dtype=torch.uint8, device=dev)
        y2 = api.wq_gemm(ad, qw, md, api.EPI_STORE_F32, ws=ws).cpu().numpy()
        assert not y2[mm:].any()
        assert np.abs(y2[:mm] - ref_b).max() <= 1e-4 * max(1.0, np.abs(ref_b).max())
        y3 = api.wq_gemm(ad, qw, md, api.EPI_STORE_F32, ws=ws).cpu().numpy()
        assert np.array_equal(y2, y3) and api.device_status() == 0


@pytest.mark.parametrize("act", [0, 1])
def test_wq_gemm_epilogues(env, act):
    api, torch, dev = env
    M, d, F, T = 200, 256, 688, 333
    bits, group = 4, 64
    a = inputs.activations(1, 11, M, d)
    m_dev = 177
    md = torch.tensor([m_dev], dtype=torch.int32, device=dev)
    # SwiGLU epilogue: gate / up rows interleaved per tile by the repack
    wq = inputs.quantized_weight(2, 12, 2 * F, d, bits, group)
    w_hat = round_act(oracle.dequantize_weight(wq), act)
    gu = oracle.linear(a[:m_dev], w_hat)
    ref = oracle.swiglu(gu[:, :F], gu[:, F:])
    qw = api.QuantWeight(wq, dev, api.ROWS_SWIGLU)
    ad = api.to_device_act(a, act, dev)
    sw = api.to_host_f32(api.wq_gemm(ad, qw, md, api.EPI_SWIGLU))
    assert sw.shape == (M, F) and not sw[m_dev:].any()
    assert np.all(np.abs(sw[:m_dev] - ref) <= np.abs(ref) * 4 * act_eps(act) + 2e-5)
    plain = api.wq_gemm(ad, qw, md, api.EPI_STORE_F32).cpu().numpy()
    assert np.abs(plain[:m_dev] - gu).max() <= 1e-4       # same weights, plain epilogue, logical columns
    # residual epilogues: u = x[idx] + a W^T (fp32), then x[idx] = bf16(u + act W_d^T)
    x = inputs.hidden_states(3, T, d)
    idx = np.sort(np.argsort(inputs.uniform(3, 5, T))[:M]).astype(np.int32)
    wo = inputs.quantized_weight(4, 13, d, d, bits, group)
    wo_hat = round_act(oracle.dequantize_weight(wo), act)
    idx_d = torch.from_numpy(idx).to(dev)
    xd = api.to_device_bf16(x, dev)
    u = api.wq_gemm(ad, api.QuantWeight(wo, dev), md, api.EPI_RESID_F32,
                    idx=idx_d, resid=xd).cpu().numpy()
    u_ref = x[idx[:m_dev]] + oracle.linear(a[:m_dev], wo_hat)
    assert np.abs(u[:m_dev] - u_ref).max() <= 1e-4 and not u[m_dev:].any()
    wd = inputs.quantized_weight(5, 14, d, F, bits, group)
    wd_hat = round_act(oracle.dequantize_weight(wd), act)
    act_in = inputs.activations(6, 15, M, F)
    u_d = torch.from_numpy(u).to(dev)
    x2 = xd.clone()
    api.wq_gemm(api.to_device_act(act_in, act, dev), api.QuantWeight(wd, dev), md, api.EPI_RESID_SCATTER,
                idx=idx_d, resid=u_d, dst=x2)
    out = api.to_host_f32(x2)
    want = u[:m_dev].astype(np.float64) + oracle.linear(act_in[:m_dev], wd_hat)
    touched = np.zeros(T, bool)
    touched[idx[:m_dev]] = True
    assert np.array_equal(out[~touched], x[~touched])     # bypass rows bit-identical
    err = np.abs(out[idx[:m_dev]] - want)
    assert np.all(err <= np.abs(want) * 2.0 ** -8 + 1e-4)
    assert api.device_status() == 0


@pytest.mark.parametrize("hd,H,Hkv,M,m_dev", [(128, 3, 1, 200, 177), (64, 3, 2, 40, None), (64, 4, 1, 300, 299)])
@pytest.mark.parametrize("act", [0, 1])
def test_wq_gemm_rotary_epilogue(env, hd, H, Hkv, M, m_dev, act):
    """QKV projection with the rotary embedding applied in the epilogue (query and key heads
    rotated at each row's position, value heads stored as they are), against the oracle's
    linear + rope.  Covers both head sizes, a head count that leaves half a row tile empty and
    all three GEMM kernels (CTA pair, single CTA, small-M)."""
    api, torch, dev = env
    d, bits, group, base = 256, 4, 64, 10000.0
    N = (H + 2 * Hkv) * hd
    a = inputs.activations(50 + hd, 11, M, d)
    wq = inputs.quantized_weight(51 + hd, 12, N, d, bits, group)
    w_hat = round_act(oracle.dequantize_weight(wq), act)
    mm = M if m_dev is None else m_dev
    pos = inputs.integers(52, 1, M, 5000)
    j = np.arange(hd // 2, dtype=np.float64)
    ang = pos[:, None].astype(np.float64) * base ** (-j / (hd // 2))
    cs = np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)        # the table is an input here
    y_ref = oracle.linear(a[:mm], w_hat)
    qk = oracle.rope(y_ref[:, :(H + Hkv) * hd], H + Hkv, hd, pos[:mm], base)
    ref = np.concatenate([qk, y_ref[:, (H + Hkv) * hd:]], axis=1)
    qw = api.QuantWeight(wq, dev, api.ROWS_ROPE64 if hd == 64 else api.ROWS_ROPE128)
    md = None if m_dev is None else torch.tensor([m_dev], dtype=torch.int32, device=dev)
    y = api.wq_gemm(api.to_device_act(a, act, dev), qw, md, api.EPI_ROPE,
                    rope_cs=torch.from_numpy(cs).to(dev), rope_features=(H + Hkv) * hd)
    assert api.device_status() == 0
    got = api.to_host_f32(y)
    assert got.shape == (M, N) and not got[mm:].any()
    # fp32 rotation of fp32 accumulators, one rounding to the activation format
    assert np.all(np.abs(got[:mm] - ref) <= np.abs(ref) * 2 * act_eps(act) + 2e-4 * max(1.0, np.abs(ref).max()))
    # the plain epilogue on the same (permuted) weights still gives the logical column order
    plain = api.wq_gemm(api.to_device_act(a, act, dev), qw, md, api.EPI_STORE_F32).cpu().numpy()
    assert np.abs(plain[:mm] - y_ref).max() <= 1e-4 * max(1.0, np.abs(y_ref).max())


@pytest.mark.parametrize("hd,H,Hkv,lens", [
    (128, 4, 2, [300, 1, 0, 128, 257]),      # ragged, an empty sequence, lengths around the tile size
    (64, 3, 3, [77, 513]),                   # 64-wide heads, five key tiles
    (128, 2, 1, [1024]),                     # eight query tiles of one sequence
    (128, 2, 2, [700, 130, 0, 520, 257]),    # sequences of 3, 1, 0, 3 and 2 blocks of 256 rows: every level of
                                             # the cost-ordered item list has a different set of sequences
])
@pytest.mark.parametrize("act", [0, 1])
def test_attention_prefill_against_oracle(env, hd, H, Hkv, lens, act):
    """Stand-alone causal attention among the executed tokens of each sequence (Eq. 3)."""
    api, torch, dev = env
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    Te = int(cu[-1])
    T_cap = Te + 70
    ld = (H + 2 * Hkv) * hd
    qkv = round_act(inputs.activations(61 + hd, 3, T_cap, ld), act)
    qkv[Te:, (H + Hkv) * hd:] = 0.0                          # value rows behind the last sequence: finite
    seq_of = np.repeat(np.arange(len(lens)), lens).astype(np.int32)
    pos = np.concatenate([np.arange(n) for n in lens]).astype(np.int32)
    ref = oracle.attention(qkv[:Te, :H * hd], qkv[:Te, H * hd:(H + Hkv) * hd], qkv[:Te, (H + Hkv) * hd:],
                           H, Hkv, hd, seq_of, pos)
    out = torch.full((T_cap, H * hd), 7.0, dtype=api.act_torch_dtype(act), device=dev)
    api.attention_prefill(api.to_device_act(qkv, act, dev), H, Hkv, hd, torch.from_numpy(cu).to(dev), act, out)
    assert api.device_status() == 0
    got = api.to_host_f32(out)
    assert np.all(got[Te:] == 7.0)                           # rows behind the executed ones untouched
    # probabilities and outputs are rounded once to the 16-bit format: a convex combination of
    # values moves by at most that rounding of the largest value, plus the output's own rounding
    vmax = np.abs(qkv[:Te, (H + Hkv) * hd:]).max()
    assert np.abs(got[:Te] - ref).max() <= 4 * act_eps(act) * vmax
    assert rel_fro(got[:Te], ref) <= 3 * act_eps(act)
    # a second call on a fresh copy of the input gives the same bits (no dependence on timing)
    out2 = torch.full((T_cap, H * hd), 7.0, dtype=api.act_torch_dtype(act), device=dev)
    api.attention_prefill(api.to_device_act(qkv, act, dev), H, Hkv, hd, torch.from_numpy(cu).to(dev), act, out2)
    assert torch.equal(out, out2)
    # the first token of a sequence sees only itself: its output is its own value row
    for b, n in enumerate(lens):
        if n:
            r = int(cu[b])
            v = qkv[r, (H + Hkv) * hd:].reshape(Hkv, hd)
            want = np.repeat(v, H // Hkv, axis=0).reshape(-1)
            assert np.array_equal(got[r], want)


def test_wq_gemm_full_size_sampled(env):
    """7B-sized gate/up projection in the launch configuration the benchmark times
    (8192-token capacity, device-side count): 66 complete output rows, two from every 256-token
    tile position of the largest tile width plus the rows around the count, against the oracle
    (every weight row tile and every K block of those token rows)."""
    api, torch, dev = env
    M, N, K, bits, group = 8192, 22016, 4096, 4, 128
    wq = inputs.quantized_weight(0, 2, N, K, bits, group)
    qw = api.QuantWeight(wq, dev)
    a = inputs.activations(7, 11, M, K)
    m_dev = 7373
    md = torch.tensor([m_dev], dtype=torch.int32, device=dev)
    y = api.wq_gemm(api.to_device_act(a, 1, dev), qw, md, api.EPI_STORE_F32)
    assert api.device_status() == 0
    off = inputs.integers(8, 1, 64, 256)
    rows = np.unique(np.concatenate([np.minimum((np.arange(64) // 2) * 256 + off, m_dev - 1),
                                     [0, 255, 256, 7371, 7372]]))
    w_hat = round_act(oracle.dequantize_weight(wq), 1)
    ref = oracle.linear(a[rows], w_hat)
    got = y[torch.from_numpy(rows).to(dev)].cpu().numpy()
    assert np.abs(got - ref).max() <= 2e-4 * max(1.0, np.abs(ref).max())
    assert not y[m_dev:].any().item()
