"""CPU-side checks of the C ABI: the library loads, exports every symbol the
header declares, validates arguments on the host, and its host-side helpers
(top-k count, offline repack) behave as documented.  No kernel is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2602_10431_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_2602_10431_b200 import build
    build.build()
    from paper_2602_10431_b200 import api as a
    a.lib()
    return a


def test_exports_every_declared_symbol(api):
    header = open(os.path.join(ROOT, "include", "qtale.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(qtale_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 14
    L = api.lib()
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert declared >= set(api.EXPORTS)


def test_strerror_and_topk_count(api):
    assert api.strerror(0) == "ok"
    for rc in range(-10, 0):
        assert api.strerror(rc) != "unknown status"
    for ratio, n in [(0.5, 256), (0.9, 8192), (0.75, 8192), (0.5, 3), (0.0, 9), (1.0, 9), (0.3333, 1000)]:
        assert api.topk_count(ratio, n) == oracle.topk_count(ratio, n)


def test_host_side_argument_validation(api):
    L = api.lib()
    n = C.c_size_t(0)
    assert L.qtale_wq_repack(None, None, None, 8, 64, 5, 64, 0, None, C.byref(n)) == -4
    assert L.qtale_wq_repack(None, None, None, 8, 64, 1, 64, 0, None, C.byref(n)) == -4
    assert L.qtale_wq_repack(None, None, None, 8, 64, 4, 32, 0, None, C.byref(n)) == -5
    assert L.qtale_wq_repack(None, None, None, 0, 64, 4, 64, 0, None, C.byref(n)) == -3
    assert L.qtale_wq_repack(None, None, None, 7, 64, 4, 64, 1, None, C.byref(n)) == -3
    assert L.qtale_wq_repack(None, None, None, 8, 64, 4, 64, 0, None, None) == -1
    # null pointers are rejected before anything is launched
    assert L.qtale_compact(None, None, None, 4, 64, None, 1e-5, 0, None, None, None) == -1
    assert L.qtale_scatter_add(None, None, None, None, None, 4, 64, None) == -1
    assert L.qtale_router_select(None, 4, 64, None, 0.0, None, None, None, 1, None, 0, 0.5, 0,
                                 None, None, None, None, None, None, 0, None) == -1
    assert L.qtale_wq_gemm(None, 64, None, 4, None, 0, 0, None, None, 64, None, 0, None) == -1
    assert L.qtale_attention_prefill(None, 384, 1, 1, 128, 1, None, 1, 8, None, 128, None) == -1
    buf = np.zeros(64, np.uint8)
    ptr = buf.ctypes.data + (-buf.ctypes.data) % 16
    # head size, head grouping, row strides and the activation format are checked before any launch
    assert L.qtale_attention_prefill(ptr, 288, 1, 1, 96, 1, ptr, 1, 8, ptr, 96, None) == -3
    assert L.qtale_attention_prefill(ptr, 640, 3, 2, 128, 1, ptr, 1, 8, ptr, 384, None) == -3
    assert L.qtale_attention_prefill(ptr, 380, 1, 1, 128, 1, ptr, 1, 8, ptr, 128, None) == -3
    assert L.qtale_attention_prefill(ptr, 384, 1, 1, 128, 7, ptr, 1, 8, ptr, 128, None) == api.lib().qtale_attention_prefill(
        ptr, 384, 1, 1, 128, 9, ptr, 1, 8, ptr, 128, None) != 0
    cfg = api.LayerConfig(256, 4, 4, 64, 688, 4, 64, 1e-5, 1e4, 0, 0.5, 1.0, 1)
    assert api.layer_workspace_bytes(cfg, 256, 2) > 256 * 256 * 2
    bad = api.LayerConfig(256, 4, 4, 48, 688, 4, 64, 1e-5, 1e4, 0, 0.5, 1.0, 1)
    assert api.layer_workspace_bytes(bad, 256, 2) == 0


@pytest.mark.parametrize("bits,group,N,K,mode", [(4, 128, 256, 256, 0), (4, 64, 200, 688, 0),
                                                 (3, 128, 128, 384, 0), (4, 64, 1376, 256, 1),
                                                 (2, 128, 256, 384, 0), (2, 64, 130, 200, 0)])
def test_repack_blob_size_and_padding(api, bits, group, N, K, mode):
    wq = inputs.quantized_weight(3, 1, N, K, bits, group)
    blob = api.wq_repack(wq["packed"], wq["scales"], wq["zeros"], N, K, bits, group, mode)
    K_pad = (K + group - 1) // group * group
    tiles = ((N // 2 + 63) // 64) if mode == 1 else (N + 127) // 128
    # row tiles are stored in pairs; every (tile, 64-wide K block) carries its codes and 128
    # (scale | zero << 16) words
    want = ((tiles + 1) // 2) * 2 * (K_pad // 64) * (128 * 64 * bits // 8 + 128 * 4)
    assert blob.nbytes == want
    # every code of the input appears in the blob: total set bits are preserved
    # for 4-bit PLAIN layouts without K padding (pure permutation of nibbles)
    if bits == 4 and mode == 0 and K == K_pad and N % 128 == 0:
        chunks = blob.reshape(-1, 4096 + 512)
        assert int(np.unpackbits(chunks[:, :4096]).sum()) == int(np.unpackbits(wq["packed"]).sum())
    if bits == 2 and K == K_pad and N % 128 == 0:     # the same for the single 2-bit plane
        chunks = blob.reshape(-1, 2048 + 512)
        assert int(np.unpackbits(chunks[:, :2048]).sum()) == int(np.unpackbits(wq["packed"]).sum())
    # too-small output buffer is reported, not overrun
    small = np.empty(16, np.uint8)
    nb = C.c_size_t(16)
    rc = api.lib().qtale_wq_repack(wq["packed"].ctypes.data, wq["scales"].view(np.uint16).ctypes.data,
                                   wq["zeros"].view(np.uint16).ctypes.data, N, K, bits, group, mode,
                                   small.ctypes.data, C.byref(nb))
    assert rc == -7
