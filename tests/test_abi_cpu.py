"""CPU-only checks of the boundary: the library builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything touches a device."""
import ctypes as C
import os
import re

import pytest

from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = C.c_void_p(0x1000)       # never dereferenced: every call below fails validation first


@pytest.fixture(scope="module")
def lib():
    build.build()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mrl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mrl_[a-z_0-9]+)\s*\(", text)))


def test_header_declarations_are_all_exported(lib):
    names = declared_functions()
    assert set(B.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in mrl.h but not exported by libmrl.so"


def test_version_and_status_strings(lib):
    assert B.version() == 104
    assert B.status_string(0) == "MRL_OK"
    assert B.status_string(4) == "MRL_ERR_WORKSPACE_TOO_SMALL"
    assert B.status_string(12345) == "MRL_ERR_UNKNOWN"


def test_workspace_bytes_is_monotone_and_aligned(lib):
    a = B.workspace_bytes(B.WS_POLICY_LOSS, 1000, 151936, 0, B.BF16, 10)
    b = B.workspace_bytes(B.WS_POLICY_LOSS, 2000, 151936, 0, B.BF16, 10)
    assert 0 < a < b and a % 256 == 0
    assert B.workspace_bytes(B.WS_TOKEN_LOGPROBS, 1000, 151936) == 0
    assert B.workspace_bytes(99, 10, 10) == 0


def test_token_logprobs_rejects_bad_arguments(lib):
    f = lib.mrl_token_logprobs
    assert f(FAKE, B.BF16, 4, 0, 8, FAKE, None, FAKE, None, None, None, 0, None) == 1       # V < 1
    assert f(FAKE, B.BF16, 4, 16, 8, FAKE, None, FAKE, None, None, None, 0, None) == 1      # ld < V
    assert f(FAKE, B.BF16, -1, 16, 16, FAKE, None, FAKE, None, None, None, 0, None) == 1    # N < 0
    assert f(None, B.BF16, 4, 16, 16, FAKE, None, FAKE, None, None, None, 0, None) == 1     # null logits
    assert f(FAKE, 7, 4, 16, 16, FAKE, None, FAKE, None, None, None, 0, None) == 3          # dtype
    assert f(None, B.BF16, 0, 16, 16, None, None, None, None, None, None, 0, None) == 0     # N = 0: no-op


def test_policy_loss_rejects_bad_arguments(lib):
    f = lib.mrl_policy_loss_fwd_bwd
    lp = B.LossParams(0.2, 0.2, 0, 0, 0.0, 0.0, 0.0, 0)

    def call(N=4, V=16, ld=16, S=1, lp_=lp, ws=FAKE, ws_bytes=1 << 20, dl=FAKE, ld_out=16, loss=FAKE, dtype=B.BF16):
        return f(FAKE, dtype, N, V, ld, FAKE, None, FAKE, S, FAKE, None, None, None,
                 C.byref(lp_) if lp_ is not None else None, dl, ld_out, None, loss, None, None, ws, ws_bytes, None)

    assert call(lp_=None) == 1
    assert call(loss=None) == 1
    assert call(V=0) == 1
    assert call(ld=8) == 1
    assert call(ld_out=8) == 1
    assert call(S=-1) == 1
    assert call(S=0) == 1                      # rows without a sequence
    assert call(dtype=5) == 3
    assert call(ws_bytes=16) == 4
    assert call(ws=None) == 4
    assert call(ws=C.c_void_p(0x1010)) == 1    # workspace not 256-byte aligned
    assert call(lp_=B.LossParams(0.2, 0.2, 9, 0, 0.0, 0.0, 0.0, 0)) == 1
    assert call(lp_=B.LossParams(-0.1, 0.2, 0, 0, 0.0, 0.0, 0.0, 0)) == 1
    # KL term: a reference trace needs somewhere to put the term and a known estimator
    assert call(lp_=B.LossParams(0.2, 0.2, 0, 0, 0.0, 0.0, 0.0, 0, None, 0x1000, 1e-3, B.KL_K3, None)) == 1
    assert call(lp_=B.LossParams(0.2, 0.2, 0, 0, 0.0, 0.0, 0.0, 0, None, 0x1000, 1e-3, 5, 0x1000)) == 1


def test_group_advantages_rejects_bad_arguments(lib):
    f = lib.mrl_group_advantages
    ap = B.AdvParams(B.ADV_GROUP_ZNORM, 0, 1e-6, 0.8, 0.2, B.PICK_SHORTEST, 0)

    def call(P=2, M=2, G=4, learner=0, ap_=ap, seq_len=FAKE, rescue=FAKE):
        return f(FAKE, seq_len, P, M, G, learner, C.byref(ap_) if ap_ is not None else None, FAKE, FAKE, rescue,
                 None, None, None, None)

    assert call(ap_=None) == 1
    assert call(M=0) == 1
    assert call(M=64, G=32) == 1               # M*G > 1024
    assert call(learner=2) == 1
    assert call(seq_len=None) == 1             # SHORTEST needs lengths
    assert call(ap_=B.AdvParams(7, 0, 1e-6, 0.8, 0.2, 0, 0)) == 1
    assert call(ap_=B.AdvParams(1, 2, 1e-6, 0.8, 0.2, 0, 0)) == 1


def test_host_pipeline_rejects_bad_arguments(lib):
    f = lib.mrl_policy_loss_fwd_bwd_host
    lp = B.LossParams(0.2, 0.2, 0, 0, 0.0, 0.0, 0.0, 0)
    cu = (C.c_int32 * 2)(0, 4)

    def call(N=4, V=16, ld=16, S=1, lp_=lp, ws=FAKE, ws_bytes=1 << 30, slab=8, loss=FAKE, dtype=B.BF16, cu_=cu):
        return f(FAKE, dtype, N, V, ld, FAKE, None, cu_, S, FAKE, None, None, None,
                 C.byref(lp_) if lp_ is not None else None, None, ld, None, loss, None, None, slab, ws, ws_bytes, None)

    assert call(lp_=None) == 1
    assert call(loss=None) == 1
    assert call(slab=0) == 1
    assert call(ld=8) == 1
    assert call(dtype=9) == 3
    assert call(V=8, ld=8) == 7                 # rows of 16 bytes: not a multiple of 32
    assert call(ws=None) == 4
    assert call(ws_bytes=64) == 4
    assert call(ws=C.c_void_p(0x1010)) == 1
    assert call(lp_=B.LossParams(0.2, 0.2, 0, B.FLAG_ACCUMULATE_LOSS, 0.0, 0.0, 0.0, 0)) == 1
    assert call(slab=3) == 7                    # the only sequence has 4 rows
    assert call(cu_=(C.c_int32 * 2)(0, 5)) == 1  # cu[S] != N
    assert lib.mrl_host_pipeline_workspace_bytes(1000, 4096, B.BF16, 8, 128) >= 3 * 128 * 4096 * 2
    assert lib.mrl_host_pipeline_workspace_bytes(1000, 4096, 9, 8, 128) == 0


def test_header_is_plain_c_and_links_from_c(tmp_path):
    """include/mrl.h compiles as C99 with pedantic warnings as errors, and a C program linked against the library
    can call the host-only entry points (no CUDA call is made)."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "abi.c"
    src.write_text('#include <stdio.h>\n#include <string.h>\n#include "mrl.h"\n'
                   "int main(void) {\n"
                   "  mrl_loss_params lp; mrl_adv_params ap; memset(&lp, 0, sizeof lp); memset(&ap, 0, sizeof ap);\n"
                   "  if (mrl_version() != MRL_VERSION) return 2;\n"
                   '  if (strcmp(mrl_status_string(MRL_OK), "MRL_OK") != 0) return 3;\n'
                   "  if (mrl_workspace_bytes(MRL_WS_POLICY_LOSS, 1000, 4096, 0, MRL_BF16, 8) == 0) return 4;\n"
                   "  if (mrl_policy_loss_fwd_bwd(0, MRL_BF16, 4, 16, 16, 0, 0, 0, 1, 0, 0, 0, 0, 0, 0, 16, 0, 0, 0, 0, 0, 0, 0)\n"
                   "      != MRL_ERR_INVALID_ARG) return 5;\n"
                   '  printf("%d %u\\n", mrl_version(), (unsigned)sizeof(mrl_loss_params));\n  return 0;\n}\n')
    exe = tmp_path / "abi"
    lib_dir = os.path.join(root, "paper_2605_07244_b200")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(root, "include"),
                    str(src), "-o", str(exe), "-L", lib_dir, "-l:libmrl.so", "-Wl,-rpath," + lib_dir], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out
    version, size = out.stdout.split()
    assert int(version) == B.version() and int(size) == C.sizeof(B.LossParams)   # the binding mirrors the C struct
