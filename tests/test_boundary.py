"""C-ABI boundary: the library loads, exports every symbol the header declares, and rejects bad
arguments before touching the GPU (no compute calls are made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2510_08431_b200 import build
    build.build_library()
    import paper_2510_08431_b200 as aj
    aj.load()
    return aj


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            src = open(os.path.join(inc, fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(attn_jvp_\w+)\s*\(", src))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2510_08431_b200 import attn_jvp
    declared = _declared_functions()
    assert {"attn_jvp_fwd", "attn_jvp_fwd_stream", "attn_jvp_device_status"} <= declared
    so = ctypes.CDLL(attn_jvp.library_path())
    for name in declared:
        assert hasattr(so, name), f"{name} is declared in include/ but not exported"
    for name in attn_jvp.EXPORTS:
        assert name in declared


def test_version_and_strerror(lib):
    assert lib.attn_jvp_version() >= 100
    assert lib.attn_jvp_strerror(0) == "ok"
    for code in range(1, 14):
        assert lib.attn_jvp_strerror(code) not in ("ok", "unknown error code")
    assert lib.attn_jvp_strerror(99) == "unknown error code"


A = 0x7F0000000000  # fake, 16-byte aligned, well separated "device" addresses (never dereferenced)
STEP = 1 << 32


def _args(**kw):
    a = dict(q=A, k=A + STEP, v=A + 2 * STEP, tq=A + 3 * STEP, tk=A + 4 * STEP, tv=A + 5 * STEP,
             o=A + 6 * STEP, to=A + 7 * STEP, lse=A + 8 * STEP, B=1, H=2, Lq=256, Lk=256, D=64, scale=0.125, flags=0)
    a.update(kw)
    return a


@pytest.mark.parametrize("kw,code", [
    (dict(flags=4), 5), (dict(flags=0x80000000), 5),
    (dict(B=0), 2), (dict(H=0), 2), (dict(Lq=0), 2), (dict(Lk=0), 2), (dict(Lk=-3), 2),
    (dict(B=1 << 20, H=1 << 20, Lq=1, Lk=1), 2),       # more work items than the kernel can index
    (dict(D=96), 3), (dict(D=0), 3), (dict(D=256), 3),
    (dict(q=None), 1), (dict(k=None), 1), (dict(v=None), 1), (dict(o=None), 1), (dict(lse=None), 1),
    (dict(tq=None), 1), (dict(to=None), 1), (dict(tk=None), 1), (dict(tv=None), 1),
    (dict(tq=None, flags=1), 1), (dict(q=None, flags=2), 1),
    (dict(scale=float("nan")), 6), (dict(scale=float("inf")), 6),
    (dict(q=A + 8), 4), (dict(o=A + 6 * STEP + 2), 4), (dict(lse=A + 8 * STEP + 4), 4), (dict(tv=A + 5 * STEP + 1), 4),
    (dict(o=A), 7), (dict(to=A + STEP + 64), 7), (dict(o=A + 7 * STEP), 7), (dict(lse=A + 2 * STEP), 7),
    (dict(o=A + 3 * STEP + 16, flags=1), 7),
])
def test_bad_arguments_are_rejected_before_any_gpu_work(lib, kw, code):
    assert lib.attn_jvp_fwd(**_args(**kw)) == code


def test_concurrent_first_calls_from_two_threads(lib):
    """The library's per-device state is set up lazily; two host threads whose first calls race must both come
    back with a clean return code.  Fake addresses: without a CUDA device the calls pass validation and stop at
    the device check, which is the lazily initialised part that can be reached here."""
    import threading
    import torch
    if torch.cuda.is_available():
        pytest.skip("would enqueue work on fake addresses")
    codes = [None] * 8
    gate = threading.Barrier(len(codes))

    def first_call(i):
        gate.wait()
        codes[i] = lib.attn_jvp_fwd(**_args()) if i % 2 == 0 else lib.attn_jvp_qknorm_fwd(
            A, A + STEP, A + 2 * STEP, A + 3 * STEP, A + 4 * STEP, 64, 64, 1e-6, None)

    threads = [threading.Thread(target=first_call, args=(i,)) for i in range(len(codes))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert all(c in (8, 9) for c in codes), codes   # ERR_ARCH / ERR_CUDA: no device; nothing crashed or hung
    assert lib.attn_jvp_device_status() == 0


def test_ignored_pointers_may_be_null_or_aliased(lib):
    """With the tangent-free / forward-only flags the unused pointers are not validated; the call then
    proceeds past validation and stops at the device check (no CUDA device here) or launches (on a GPU machine
    this test is skipped so that nothing is enqueued on fake addresses)."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("would enqueue work on fake addresses")
    for kw in (dict(tk=None, tv=None, flags=1), dict(tq=None, tk=None, tv=None, to=None, flags=2),
               dict(tk=A + 6 * STEP, tv=A + 8, flags=1)):
        rc = lib.attn_jvp_fwd(**_args(**kw))
        assert rc in (8, 9), rc  # ERR_ARCH / ERR_CUDA: validation passed, no device


def test_python_wrapper_validates_tensors(lib):
    import torch
    q = torch.zeros(1, 8, 2, 64, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        lib.attention_jvp(q, q, q, q, q, q)  # CPU tensors are refused: there is no CPU path


def test_workspace_size_functions_are_plain_host_arithmetic(lib):
    """Sizes of the two caller-provided workspaces (no GPU involved)."""
    # split-KV: per chunk fp32 O and tO partials [B][Lq][H][D] and fp32 LSE, mu partials [B][H][Lq] (16-byte padded)
    B, H, Lq, Lk, D = 1, 8, 512, 32760, 128
    assert lib.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, 1) == 0          # one chunk: the plain kernel
    four = lib.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, 4)
    assert four == 2 * 4 * B * Lq * H * D * 4 + 2 * 4 * B * H * Lq * 4
    assert lib.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, 96, 4) == 0
    # host pipeline: three buffer sets of one head group (default: sized for five stages' worth of heads) (4 Q-side + 4 K-side bf16 tensors + LSE, 256-byte padded)
    pad = lambda n: (n + 255) // 256 * 256
    for (B, H, Lq, Lk, D, hps, hg) in ((1, 40, 32760, 32760, 128, 0, 8), (1, 40, 32760, 32760, 128, 3, 3),
                                       (2, 5, 300, 200, 128, 2, 2), (1, 7, 129, 513, 64, 0, 4),
                                       (1, 3, 50, 60, 64, 0, 3), (1, 2, 50, 60, 128, 9, 2)):
        want = 3 * (4 * pad(B * Lq * hg * D * 2) + 4 * pad(B * Lk * hg * D * 2) + pad(B * hg * Lq * 4))
        assert lib.attn_jvp_host_workspace_bytes(B, H, Lq, Lk, D, hps) == want
    assert lib.attn_jvp_host_workspace_bytes(1, 4, 64, 64, 96, 0) == 0
    assert lib.attn_jvp_host_workspace_bytes(1, 4, 64, 64, 64, -1) == 0


def test_host_entry_point_rejects_bad_arguments_before_any_gpu_work(lib):
    """attn_jvp_fwd_host validates everything, including the workspace, before it creates a stream or copies."""
    base = [A, A + STEP, A + 2 * STEP, A + 3 * STEP, A + 4 * STEP, A + 5 * STEP, A + 6 * STEP, A + 7 * STEP,
            A + 8 * STEP, 1, 4, 128, 128, 128, 0.088, 0, 0]
    need = lib.attn_jvp_host_workspace_bytes(1, 4, 128, 128, 128, 0)
    ws = A + 9 * STEP

    def call(args, workspace=ws, nbytes=need):
        return lib.attn_jvp_fwd_host(*args, workspace, nbytes, None)

    assert call(base, nbytes=need - 1) == 12
    assert call(base, workspace=ws + 16) == 4
    assert call(base, workspace=None) == 1
    for idx, val, code in ((0, None, 1), (3, None, 1), (7, None, 1), (8, None, 1), (15, 0x10, 5), (16, -2, 2),
                           (9, 0, 2), (13, 80, 3), (14, float("nan"), 6)):
        bad = list(base)
        bad[idx] = val
        assert call(bad) == code, (idx, val)


def test_suggest_splits_is_one_without_a_device_or_for_bad_shapes(lib):
    import torch
    assert lib.attn_jvp_suggest_splits(1, 8, 512, 32760, 96) == 1
    assert lib.attn_jvp_suggest_splits(0, 8, 512, 32760, 128) == 1
    if not torch.cuda.is_available():
        assert lib.attn_jvp_suggest_splits(1, 8, 512, 32760, 128) == 1
