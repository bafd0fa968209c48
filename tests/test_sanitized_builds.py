"""The two stand-ins for a device memory checker.

* Host logic (argument validation, Eq. 1 layout, Eq. 3 schedule, schedule dump, closed-form counts) compiled with
  -fsanitize=address,undefined and driven through the C ABI in a child process that preloads the sanitizer runtime:
  any out-of-bounds access or undefined arithmetic in it aborts the child.  Needs no GPU.
* The KSA_DEBUG build of the kernels (every global output index is checked against its tensor, a status code is
  recorded and the access skipped instead of made) on the small edge shapes, against the oracle.  Needs the GPU.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

HOST_SCRIPT = r"""
import sys
sys.path.insert(0, %(root)r)
from paper_2604_24432_b200 import binding as ksa
shapes = [([1], 8, 1, 2, 2, 2, 64), ([7], 8, 1, 2, 2, 1, 128), ([127, 129, 128], 8, 1, 3, 4, 2, 64),
          ([333, 1000], 3, 2, 5, 6, 2, 128), ([777], 16, 0, 7, 4, 4, 64), ([640], 1, 1, 100, 2, 1, 128),
          ([1290], 200, 3, 1, 4, 1, 128), ([2048, 640, 1336], 8, 1, 16, 8, 2, 128), ([1280], 128, 128, 1, 4, 2, 128),
          ([8192], 8, 1, 128, 32, 8, 128), ([48729, 62038, 9062], 64, 8, 16, 32, 8, 128)]
n = 0
for lens, k, m, C, Hq, Hkv, D in shapes:
    p = ksa.Problem(lens, k, m, C, Hq, Hkv, D, 0.1)
    n += len(ksa.schedule_dump(p)) + ksa.visible_pairs(p) %% 7 + ksa.workspace_bytes(p) %% 3 + ksa.total_aug_len(p) %% 5
    n += len(ksa.position_ids(p)) %% 3 if hasattr(ksa, "position_ids") else 0
for bad in (dict(k=0), dict(m=-1), dict(C=-1), dict(Hq=3), dict(D=96), dict(text_lens=[10, 0, 5]), dict(flags=0x80)):
    kw = dict(text_lens=[100], k=8, m=1, C=2, Hq=4, Hkv=2, D=64, scale=0.125); kw.update(bad)
    try:
        ksa.workspace_bytes(ksa.Problem(**kw))
        raise SystemExit("accepted " + repr(bad))
    except ksa.KsaError:
        pass
print("host logic ok", n)
"""


def test_host_logic_under_address_and_undefined_behaviour_sanitizers():
    from paper_2604_24432_b200 import build as ksa_build
    ksa_build.build(variant="asan")
    asan = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    ubsan = subprocess.run(["gcc", "-print-file-name=libubsan.so"], capture_output=True, text=True).stdout.strip()
    if not (os.path.isabs(asan) and os.path.exists(asan)):
        pytest.skip("no sanitizer runtime beside gcc")
    env = dict(os.environ, KSA_B200_LIB_VARIANT="asan", LD_PRELOAD=asan + (":" + ubsan if os.path.exists(ubsan) else ""),
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=1:protect_shadow_gap=0", UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    r = subprocess.run([sys.executable, "-c", HOST_SCRIPT % dict(root=ROOT)], capture_output=True, text=True, env=env, timeout=900)
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])
    assert "host logic ok" in r.stdout
    assert "AddressSanitizer" not in r.stderr and "runtime error" not in r.stderr, r.stderr[-3000:]


DEBUG_SCRIPT = r"""
import sys
sys.path.insert(0, %(root)r)
from paper_2604_24432_b200 import binding as ksa, synth
from tests import parity
assert ksa.LIB_PATH.endswith("_debug.so")
ctx = ksa.Context(0)
shapes = [([1], 8, 1, 2, 2, 2, 64), ([7], 8, 1, 2, 2, 1, 128), ([127, 129, 128], 8, 1, 3, 4, 2, 64),
          ([333, 1000], 3, 2, 5, 6, 2, 128), ([777], 16, 0, 7, 4, 4, 64), ([640], 1, 1, 100, 2, 1, 128),
          ([1290], 200, 3, 1, 4, 1, 128), ([2100], 8, 1, 16, 8, 2, 128), ([2048, 640, 1336], 8, 1, 16, 8, 2, 128),
          ([1024, 320], 4, 2, 9, 4, 2, 64), ([768], 128, 1, 2, 2, 1, 128), ([1300], 200, 8, 1, 8, 1, 128)]
for flags in (0, ksa.KSA_FLAG_REFERENCE_KERNEL, ksa.KSA_FLAG_CTA_PAIR_KERNEL):
    for lens, k, m, C, Hq, Hkv, D in shapes:
        wl = synth.Workload("dbg", 99, lens, Hq, Hkv, D)
        parity.check_workload(ctx, wl, synth.Layout("dbg", k, m, C), flags)     # asserts the status word is 0
print("debug build ok")
"""


@pytest.mark.gpu
def test_debug_build_edge_shapes():
    from paper_2604_24432_b200 import build as ksa_build
    ksa_build.build(variant="debug")
    env = dict(os.environ, KSA_B200_LIB_VARIANT="debug")
    r = subprocess.run([sys.executable, "-c", DEBUG_SCRIPT % dict(root=ROOT)], capture_output=True, text=True, env=env, timeout=1500, cwd=ROOT)
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])
    assert "debug build ok" in r.stdout
