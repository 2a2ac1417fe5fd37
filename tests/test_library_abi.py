"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, and validates descriptors before touching the device."""
import ctypes as C
import os
import re

import pytest

import paper_2211_00188_b200 as pkg
from paper_2211_00188_b200 import binding as B
from paper_2211_00188_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    builder.build()
    return pkg.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "adacgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adacgd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 10
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(pkg.EXPORTED_SYMBOLS) == names


def problem(n=4, d=100, loss=B.LOSS_NONE):
    return B._Problem(loss, 0.0, n, 0, d, 0, None, None, None, None, None, 0)


def ws_bytes(lib, prob, worker, master=(), zeta=1.0):
    w, k1 = B._cset(worker, zeta)
    m, k2 = B._cset(master, zeta)
    out = C.c_size_t(0)
    st = lib.adacgd_workspace_bytes(C.byref(prob), C.byref(w), C.byref(m), 0, C.byref(out))
    return st, out.value, lib.adacgd_last_error(None).decode()


def test_workspace_bytes_and_descriptor_validation(lib):
    st, nbytes, _ = ws_bytes(lib, problem(), [(B.TOPK, 5), (B.TOPK, 50)])
    assert st == 0 and nbytes > 0
    st2, nbytes2, _ = ws_bytes(lib, problem(n=8, d=100000), [(B.TOPK, 5)])
    assert st2 == 0 and nbytes2 > nbytes
    # Top-K parameters must increase (strongest compression first, Section 4.3)
    st, _, msg = ws_bytes(lib, problem(), [(B.TOPK, 50), (B.TOPK, 5)])
    assert st == 2 and "increasing" in msg
    st, _, msg = ws_bytes(lib, problem(), [(B.QUANT, 8), (B.QUANT, 4)])
    assert st == 2
    st, _, msg = ws_bytes(lib, problem(), [(B.TOPK, 0)])
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(), [(B.QUANT, 1)])
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(), [(B.QUANT, 17)])
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(), [(7, 3)])
    assert st == 1 and "kind" in msg
    st, _, msg = ws_bytes(lib, problem(), [(B.TOPK, 5)], zeta=-1.0)
    assert st == 1 and "zeta" in msg
    st, _, msg = ws_bytes(lib, problem(), [(B.TOPK, 5)], zeta=float("nan"))
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(n=0), [(B.TOPK, 5)])
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(d=0), [(B.TOPK, 5)])
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(d=2 ** 31), [(B.TOPK, 5)])
    assert st == 1
    st, _, msg = ws_bytes(lib, problem(), [(B.TOPK, i + 1) for i in range(9)])
    assert st == 1
    # a dense objective without data pointers
    st, _, msg = ws_bytes(lib, B._Problem(0, 0.1, 4, 0, 100, 10, None, None, None, None, None, 0), [(B.TOPK, 5)])
    assert st == 1 and "A" in msg
    # two identity-or-wider Top-K candidates cannot both be last
    st, _, msg = ws_bytes(lib, problem(d=100), [(B.TOPK, 100), (B.TOPK, 200)])
    assert st == 2


def test_null_arguments_are_rejected_without_a_device(lib):
    assert lib.adacgd_workspace_bytes(None, None, None, 0, None) == 1
    ctx = C.c_void_p()
    assert lib.adacgd_init(C.byref(ctx), None, None, None, None, 1.0, 1, 0, None, 0, None) == 1
    assert not ctx.value
    assert lib.adacgd_step(None, 1, None, None) == 1
    assert lib.adacgd_get_state(None, 0, None, 0, 0) == 1
    assert lib.adacgd_launch_count(None) == 0
    lib.adacgd_destroy(None)
    assert isinstance(lib.adacgd_last_error(None), bytes)


def test_init_rejects_small_or_misaligned_workspace(lib):
    prob = problem()
    w, k = B._cset([(B.TOPK, 5)], 1.0)
    ctx = C.c_void_p()
    st = lib.adacgd_init(C.byref(ctx), C.byref(prob), C.byref(w), None, None, 1.0, 1, 0, C.c_void_p(256), 16, None)
    assert st == 4
    st = lib.adacgd_init(C.byref(ctx), C.byref(prob), C.byref(w), None, None, 1.0, 1, 0, C.c_void_p(8), 1 << 30, None)
    assert st == 1


def test_binding_fails_loudly_without_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    with pytest.raises(RuntimeError):
        pkg.AdaCGD(2, 10, [(pkg.TOPK, 1)], 1.0)


def test_message_bits_is_exported_and_matches_the_oracle_formula(lib):
    from oracle import adacgd_oracle as O
    for d in (1, 2, 3, 8, 9, 1000, 1024, 1025, 25_000_000, 2 ** 31 - 1):
        for cand in [(B.TOPK, 1), (B.TOPK, 7), (B.TOPK, d), (B.TOPK, d + 5), (B.QUANT, 2), (B.QUANT, 8), (B.QUANT, 16)]:
            assert B.message_bits(cand, d) == O.message_bits(cand, d), (cand, d)
    # invalid descriptors give 0, not a crash
    assert B.message_bits((B.TOPK, 0), 10) == 0 and B.message_bits((B.QUANT, 1), 10) == 0
    assert B.message_bits((9, 3), 10) == 0 and B.message_bits((B.TOPK, 3), 0) == 0
    assert lib.adacgd_message_bits(None, 10) == 0


def test_init_without_a_device_names_the_failing_call(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    prob = problem()
    w, k = B._cset([(B.TOPK, 5)], 1.0)
    nbytes = C.c_size_t(0)
    assert lib.adacgd_workspace_bytes(C.byref(prob), C.byref(w), None, 0, C.byref(nbytes)) == 0
    ctx = C.c_void_p()
    st = lib.adacgd_init(C.byref(ctx), C.byref(prob), C.byref(w), None, None, 1.0, 1, 0, C.c_void_p(4096), nbytes.value, None)
    assert st == 5 and not ctx.value                       # ADACGD_ERR_CUDA, no context handed out
    msg = lib.adacgd_last_error(None).decode()
    assert msg.startswith("adacgd_init (") and ":" in msg, msg   # which call failed, then the runtime's reason
