"""The C-ABI library: it loads, exports every function the header declares, and rejects bad
arguments on the host before touching the device (so these run without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2410_15651_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(rlhf_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported_and_bound(lib):
    declared = _declared()
    assert {"rlhf_gather_logprobs", "rlhf_kl_reward", "rlhf_gae", "rlhf_ppo_loss_fwd_bwd"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.SIGNATURES), declared ^ set(binding.SIGNATURES)


def test_status_strings(lib):
    assert lib.rlhf_status_string(0) == b"RLHF_OK"
    assert lib.rlhf_status_string(5) == b"RLHF_ERR_WORKSPACE"
    assert lib.rlhf_status_string(16) == b"RLHF_ERR_ID_RANGE"
    assert lib.rlhf_status_string(16 | 64) == b"RLHF_ERR_ID_RANGE|RLHF_ERR_TIMEOUT"
    assert lib.rlhf_status_string(12345) == b"RLHF_ERR_UNKNOWN"


def test_workspace_size_is_linear_in_tokens(lib):
    assert lib.rlhf_workspace_bytes(0, 5) == 0 and lib.rlhf_workspace_bytes(3, -1) == 0
    for B, T in ((2, 16), (16, 256), (128, 1024)):
        n = lib.rlhf_workspace_bytes(B, T)
        assert n % 256 == 0 and 4 * B * T <= n <= 16 * B * T + 65536


def test_host_side_argument_checks(lib):
    buf = (ctypes.c_char * 65536)()
    base = ctypes.addressof(buf)
    p = (base + 255) // 256 * 256           # a 256-byte aligned host address: never dereferenced
    ws_n = lib.rlhf_workspace_bytes(2, 4)
    # step 1
    ok = dict(logits=p, sb=32, st=8, ids=p, isb=4, lengths=p, B=2, T=4, V=8, out=p, ws=p, wsn=ws_n, stream=None)

    def s1(**kw):
        a = dict(ok, **kw)
        return lib.rlhf_gather_logprobs(a["logits"], a["sb"], a["st"], a["ids"], a["isb"], a["lengths"],
                                        a["B"], a["T"], a["V"], a["out"], a["ws"], a["wsn"], a["stream"])

    assert s1(logits=None) == 1 and s1(out=None) == 1 and s1(ws=None) == 1
    assert s1(B=0) == 2 and s1(V=-3) == 2
    assert s1(ids=p + 4) == 3 and s1(ws=p + 16) == 3
    assert s1(st=7) == 4 and s1(sb=-1) == 4
    assert s1(wsn=ws_n - 1) == 5
    # steps 2 and 3
    assert lib.rlhf_kl_reward(p, p, p, p, 2, 4, -0.1, 5.0, p, None) == 6
    assert lib.rlhf_kl_reward(p, p, p, p, 2, 4, 0.1, float("nan"), p, None) == 6
    assert lib.rlhf_kl_reward(p, None, p, p, 2, 4, 0.1, 5.0, p, None) == 1
    assert lib.rlhf_gae(p, p + 64, p, 2, 4, 1.5, 0.9, p + 128, p + 192, None) == 6
    assert lib.rlhf_gae(p, p + 64, p, 2, 4, 0.9, 0.9, p, p + 192, None) == 4       # output aliases input
    # step 4
    def s4(**kw):
        a = dict(logits=p, sb=32, st=8, ids=p, isb=4, lengths=p, f=p, B=2, T=4, V=8, eps=0.2, vclip=0.2,
                 gs=1.0, loss=p, dl=p + 1024, dsb=32, dst=8, dv=p, lpn=None, ws=p, wsn=ws_n)
        a.update(kw)
        return lib.rlhf_ppo_loss_fwd_bwd(a["logits"], a["sb"], a["st"], a["ids"], a["isb"], a["lengths"],
                                         a["f"], a["f"], a["f"], a["f"], a["f"], a["B"], a["T"], a["V"],
                                         a["eps"], a["vclip"], a["gs"], a["loss"], a["loss"],
                                         a["dl"], a["dsb"], a["dst"], a["dv"], a["lpn"], a["ws"], a["wsn"], None)

    assert s4(dl=None) == 1 and s4(f=None) == 1
    assert s4(eps=0.0) == 6 and s4(eps=1.0) == 6 and s4(gs=float("inf")) == 6 and s4(vclip=-1.0) == 6
    assert s4(dst=7) == 4 and s4(dsb=24) == 4                # rows too close / sequences overlapping
    assert s4(dl=p, dsb=64) == 4                             # in place needs equal strides
    assert s4(wsn=100) == 5
    # B*T above 2^29 is refused (the log-prob kernel walks up to 2*B*T rows with 32-bit indices)
    big = lib.rlhf_workspace_bytes(1 << 15, 1 << 14)
    assert s1(B=1 << 15, T=1 << 14, wsn=big - 256) == 5      # exactly 2^29 passes the shape check (the workspace is checked next)
    assert s1(B=(1 << 15) + 1, T=1 << 14) == 2
    assert s4(B=(1 << 15) + 1, T=1 << 14) == 2
    assert lib.rlhf_kl_reward(p, p, p, p, (1 << 15) + 1, 1 << 14, 0.1, 5.0, p, None) == 2
    # whitening
    assert lib.rlhf_whiten_advantages(None, p, 2, 4, 1e-8, p, p, ws_n, None) == 1
    assert lib.rlhf_whiten_advantages(p, p, 2, 4, -1.0, p, p, ws_n, None) == 6
    assert lib.rlhf_whiten_advantages(p, p, 2, 4, float("inf"), p, p, ws_n, None) == 6
    assert lib.rlhf_whiten_advantages(p, p, 2, 4, 1e-8, p, p, 8, None) == 5
    assert lib.rlhf_whiten_advantages(p, p, 0, 4, 1e-8, p, p, ws_n, None) == 2
    # bounded-wait self-test: limit must be positive and at most 2 s
    assert lib.rlhf_selftest_bounded_wait(None, ws_n, 1000, None) == 1
    assert lib.rlhf_selftest_bounded_wait(p, ws_n, 0, None) == 6
    assert lib.rlhf_selftest_bounded_wait(p, ws_n, 3 * 10 ** 9, None) == 6
    assert lib.rlhf_selftest_bounded_wait(p, 100, 1000, None) == 5


def test_binding_refuses_cpu_tensors():
    import torch
    z = torch.zeros((1, 2, 8), dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        binding.gather_logprobs(z, torch.zeros((1, 2), dtype=torch.int64), torch.ones(1, dtype=torch.int32),
                                torch.zeros(8192, dtype=torch.uint8))


@pytest.mark.parametrize("n_valid,n_padded,G", [(3006, 1090, 148), (0, 77, 148), (5, 0, 148), (148, 148, 148),
                                                (9228, 7156, 148), (42800, 88272, 148), (7, 3, 4), (1000, 1, 148),
                                                (149, 500, 148), (147, 293, 148)])
def test_pad_share_tiles_the_padded_rows_and_balances_bytes(lib, n_valid, n_padded, G):
    shares = [binding.pad_share(n_valid, n_padded, G, i) for i in range(G)]
    # contiguous, in block order, covering [0, n_padded) exactly once
    pos = 0
    for start, count in shares:
        assert start == pos and count >= 0
        pos += count
    assert pos == n_padded
    # cost in units of one row written: a valid row counts 2 (read + write), a padded row 1
    rows = [n_valid // G + (1 if i < n_valid % G else 0) for i in range(G)]
    cost = [2 * r + c for r, (_, c) in zip(rows, shares)]
    if n_padded >= 2 * (G - n_valid % G):
        assert max(cost) - min(cost) <= 1               # enough padded rows to level the blocks
    else:
        # too few to level: they all go to the blocks with one valid row fewer, spread evenly
        assert all(c == 0 for (_, c), r in zip(shares, rows) if r == max(rows) and max(rows) != min(rows))
        lows = [c for (_, c), r in zip(shares, rows) if r == min(rows)]
        assert max(lows) - min(lows) <= 1


def test_pad_share_rejects_bad_arguments(lib):
    s, c = ctypes.c_longlong(), ctypes.c_longlong()
    assert lib.rlhf_pad_share(1, 1, 0, 0, ctypes.byref(s), ctypes.byref(c)) == 2
    assert lib.rlhf_pad_share(1, 1, 4, 4, ctypes.byref(s), ctypes.byref(c)) == 2
    assert lib.rlhf_pad_share(-1, 1, 4, 0, ctypes.byref(s), ctypes.byref(c)) == 2
    assert lib.rlhf_pad_share(1, 1, 4, 0, None, ctypes.byref(c)) == 1
