"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, sizes its workspace sensibly and rejects bad arguments
before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2602_19362_b200 import binding as B, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return B.lib()


def _problem(**kw):
    p = B.OaplProblem()
    p.N, p.d, p.V, p.S, p.P = 1024, 256, 4096, 16, 4
    for f in ("H", "W", "targets", "mask", "seq_id", "group_id", "reward", "logp_inf"):
        setattr(p, f, 0x1000)                    # fake, aligned, never dereferenced on these paths
    p.beta_v = p.beta_loss = p.loss_scale = 1.0
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "oapl.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(oapl_[a-z_]+)\s*\(", header))
    assert {"oapl_token_logprobs", "oapl_value_estimate", "oapl_loss_fwd", "oapl_loss_bwd"} <= declared
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(B.EXPORTS)


def test_workspace_size(L):
    w = lambda **kw: B.oapl_workspace_bytes(_problem(**kw))
    assert w() > 0
    assert w(N=0) == 0 and w(d=100) == 0 and w(V=0) == 0 and w(S=0) == 0
    # linear in N for fixed V (row-chunk of logit gradients is bounded), never ~ N*V
    big, bigger = w(N=1 << 20, d=1024, V=150000), w(N=1 << 21, d=1024, V=150000)
    assert bigger - big < 1.05 * (1 << 20) * (2 * 1024 + 4 * 6 + 12 * 16 + 8)
    assert bigger < 0.02 * (1 << 21) * 150000 * 2


def test_argument_errors_return_before_any_device_work(L):
    ws, n = ctypes.c_void_p(0x10000), 1 << 40
    st = ctypes.c_void_p(0)
    out = ctypes.c_void_p(0x2000)
    call = lambda p: L.oapl_loss_fwd(ctypes.byref(p), out, out, out, None, None, ws, n, 0, st)
    assert L.oapl_loss_fwd(None, out, out, out, None, None, ws, n, 0, st) == -1
    assert call(_problem(d=96)) == -4
    assert call(_problem(N=-5)) == -1
    assert call(_problem(beta_v=0.0)) == -1
    assert call(_problem(beta_loss=float("nan"))) == -1
    assert call(_problem(beta_loss=float("inf"))) == -1
    assert call(_problem(H=0)) == -1
    assert call(_problem(H=0x1008)) == -2
    assert call(_problem(reward=0)) == -1
    p = _problem()
    assert L.oapl_loss_fwd(ctypes.byref(p), None, out, out, None, None, ws, n, 0, st) == -1
    assert L.oapl_loss_fwd(ctypes.byref(p), out, out, out, None, None, ctypes.c_void_p(0x10010), n, 0, st) == -2
    assert L.oapl_loss_fwd(ctypes.byref(p), out, out, out, None, None, ws, 1000, 0, st) == -3
    assert L.oapl_loss_bwd(ctypes.byref(p), None, out, 0, ws, n, 0, st) == -1
    assert L.oapl_loss_bwd(ctypes.byref(p), ctypes.c_void_p(0x2004), out, 0, ws, n, 0, st) == -2
    assert L.oapl_token_logprobs(ctypes.byref(p), None, None, ws, n, 0, st) == -1
    assert L.oapl_value_estimate(out, out, 8, 2, -1.0, out, st) == -1
    assert L.oapl_value_estimate(None, out, 8, 2, 1.0, out, st) == -1
    assert L.oapl_debug_gemm(out, out, out, 128, 256, 100, 0, 0, 0, 0, 0, out, st) == -4
    assert L.oapl_debug_gemm(out, out, out, 128, 256, 128, 0, 0, 0, 0, 0, None, st) == -1
    # leaving a pipeline step out needs a short wait limit
    assert L.oapl_debug_gemm(out, out, out, 128, 256, 128, 0, 0, 0, 0, 3, out, st) == -1
    assert L.oapl_debug_gemm(out, out, out, 128, 256, 128, 0, 0, 0, 10 ** 9, 3, out, st) == -1
    # the single call with options: negative bounds
    opt = B.OaplCallOptions()
    opt.live_rows_bound = -1
    args = (out, out, out, None, None, out, out, 0, ws, n, 1)
    assert L.oapl_loss_fwd_bwd_ex(ctypes.byref(p), *args, ctypes.byref(opt), st) == -1
    opt.live_rows_bound, opt.max_seq_rows_bound = 100, -7
    assert L.oapl_loss_fwd_bwd_ex(ctypes.byref(p), *args, ctypes.byref(opt), st) == -1


def test_workspace_free_entry_point_rejects_sizes_beyond_its_built_in_scratch(L):
    # N <= 2048, d <= 1024, S <= 2048: refused on the host, before any CUDA call
    st, out = ctypes.c_void_p(0), ctypes.c_void_p(0x2000)
    call = lambda p: L.oapl_token_logprobs_static(ctypes.byref(p), out, None, None, st)
    assert call(_problem(N=2049)) == -4
    assert call(_problem(d=1088)) == -4
    assert call(_problem(N=2048, S=2049)) == -4
    assert call(_problem(d=100)) == -4
    assert L.oapl_token_logprobs_static(ctypes.byref(_problem()), None, None, None, st) == -1


def test_contraction_timing_applies_only_on_the_device_it_was_enabled_on(L):
    # host logic only: a launch is timed (and given the device counters' address) only when the
    # current device is the one the timing was enabled on
    assert L.oapl_profile_applies(-1, 0) == 0
    assert L.oapl_profile_applies(0, 0) == 1
    assert L.oapl_profile_applies(0, 1) == 0
    assert L.oapl_profile_applies(3, 3) == 1
    assert L.oapl_profile_applies(3, 0) == 0


def test_range_slot_bound_covers_the_greedy_packing(L):
    # the single call enqueues oapl_range_slots(...) slots without knowing the ranges; the greedy
    # packing of whole sequences (close a range when the next sequence does not fit) must never
    # need more, with and without the bound on the longest sequence
    import random
    rnd = random.Random(0)
    for trial in range(400):
        stage = rnd.choice([256, 512, 4096, 32768])
        S = rnd.randint(1, 200)
        longest = rnd.randint(1, stage)
        lens = [rnd.randint(0, longest) if rnd.random() < 0.9 else 0 for _ in range(S)]
        if rnd.random() < 0.3:
            lens = [longest if rnd.random() < 0.7 else 1 for _ in range(S)]   # adversarial: long, short, long
        n, cur = 0, -1
        for l in lens:
            if l == 0:
                continue
            if cur < 0:
                cur = 0
            if cur + l > stage:
                n += 1
                cur = 0
            cur += l
        n += 1 if cur >= 0 else 0
        live = sum(lens)
        assert n <= L.oapl_range_slots(live, max(lens), stage, S), (lens, stage)
        assert n <= L.oapl_range_slots(live, 0, stage, S), (lens, stage)
        assert n <= L.oapl_range_slots(live + 5000, 0, stage, S)
    # the 7B-scale benchmark batch: 309040 response tokens, sequences up to 4096
    assert L.oapl_range_slots(309040, 4096, 65536, 128) == 6
    assert L.oapl_range_slots(309040, 4096, 32768, 128) == 11
    assert L.oapl_range_slots(524288, 0, 32768, 128) == 31
    assert L.oapl_range_slots(10, 0, 32768, 128) == 1
    assert L.oapl_range_slots(-1, 0, 32768, 128) == -1


def test_status_strings(L):
    for code in range(0, -14, -1):
        assert L.oapl_status_string(code) not in (None, b"unknown status")
    assert L.oapl_status_string(-99) == b"unknown status"


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "liboapl.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()
