"""The oracle under AddressSanitizer and UndefinedBehaviorSanitizer.

The oracle is the yardstick for every parity test, so a read or write past one of its arrays would
silently move the yardstick.  It is compiled once more with -fsanitize=address,undefined and every
function is driven, in a child process, over sizes chosen to sit on and next to every boundary
(one entry, a chunk, a chunk plus and minus one, short last chunks, k = 0 and k = d).  numpy's
arrays come from malloc, which the sanitizer surrounds with red zones, so an access one element
outside any argument array ends the child with a report."""
import os
import shutil
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

DRIVER = textwrap.dedent("""
    import sys
    import numpy as np
    sys.path.insert(0, sys.argv[2])
    import oracle
    oracle._lib = oracle.load(sys.argv[1])          # every call below runs the sanitized build
    Q = oracle.QSpec
    r = np.random.default_rng(0)
    for d in (1, 3, 4, 5, 31, 32, 33, 127, 128, 129, 255, 256, 257, 1000, 4095, 4096, 4097):
        v = (r.standard_normal(d) * 10.0 ** r.uniform(-3, 3)).astype(np.float32)
        v[r.integers(0, d)] = 0.0
        oracle.q_ternary(v, 2**40 + 3, 7, 2)
        c, p = oracle.q_ternary(v, 5, 1, oracle.SERVER_WID)
        oracle.decode_ternary(p["sgn"], p["nz"], p["scale"], d)
        for L in (0, 4, 128, 256, 4096):
            oracle.q_sign1(v, L, 1); oracle.q_sign1(v, L, 2)
            c, p = oracle.q_sign1(v, L)
            oracle.decode_sign1(p["bits"], p["scale"], d, L)
            for s in ((1, 15, 255) if L else ()):
                c, p = oracle.q_qsgd(v, L, s, 2**40 + 3, 7, 2)
                oracle.decode_qsgd(p["lvl"], p["sgn"], p["step"], d, L)
            for S in ((2, 4) if L else ()):
                for scaled in (0, 1):
                    c, p = oracle.q_rsparse(v, L, S, scaled, 5, 1, 0)
                    oracle.decode_rsparse(p["val"], p["off"], d, L, S)
        for k in sorted({0, 1, d // 2, max(d - 1, 0), d}):
            c, p = oracle.q_topk(v, k)
            oracle.decode_topk(p["idx"], p["val"], d)
        for b in (16, 24):
            c, p = oracle.q_clip(v, b)
            oracle.decode_clip(p["hi"], d, b)
        oracle.q_identity(v)
    for n in (1, 2, 128):
        oracle.pairwise_sum(r.standard_normal(n).astype(np.float32))
    oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    ops = [Q("identity"), Q("ternary"), Q("sign1", chunk=0), Q("sign1", chunk=128), Q("sign1", chunk=128, norm=2), Q("topk", k=17), Q("qsgd", chunk=128, levels=15),
           Q("clip", bits=16), Q("clip", bits=24), Q("rsparse", chunk=128, keep_one_in=4)]
    for wq in ops:
        for sq in ops:
            n, d = 3, 333
            st = oracle.State.zeros(n, d)
            for t in range(2):
                oracle.step(st, r.standard_normal((n, d)).astype(np.float32), wq, sq, 0.1, 9, t, compensate=bool(t))
    print("sanitized oracle ok")
""")


def test_oracle_is_clean_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    libasan = subprocess.run([gcc, "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    if not os.path.isabs(libasan) or not os.path.exists(libasan):
        pytest.skip("gcc has no libasan here")
    so = str(tmp_path / "libdsq_oracle_san.so")
    subprocess.run([gcc, "-std=c11", "-O1", "-g", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
                    "-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer",
                    "-o", so, os.path.join(ROOT, "oracle", "dsq_oracle.c"), "-lm"], check=True)
    env = dict(os.environ, LD_PRELOAD=libasan, ASAN_OPTIONS="detect_leaks=0:abort_on_error=0:halt_on_error=1",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    run = subprocess.run([sys.executable, "-c", DRIVER, so, ROOT], capture_output=True, text=True, env=env, timeout=600)
    assert run.returncode == 0 and "sanitized oracle ok" in run.stdout, (run.stdout[-2000:], run.stderr[-4000:])


def test_the_sanitizer_setup_does_catch_an_overrun(tmp_path):
    """The same harness on a deliberately broken copy of the oracle (the sign words written one word
    too far): the child must fail, which shows that a clean run above means something."""
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    libasan = subprocess.run([gcc, "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    if not os.path.isabs(libasan) or not os.path.exists(libasan):
        pytest.skip("gcc has no libasan here")
    src = open(os.path.join(ROOT, "oracle", "dsq_oracle.c")).read()
    broken = src.replace("memset(bits, 0, sizeof(uint32_t) * nw);", "memset(bits, 0, sizeof(uint32_t) * (nw + 1));", 1)
    assert broken != src
    csrc, so = str(tmp_path / "broken.c"), str(tmp_path / "libbroken.so")
    open(csrc, "w").write(broken)
    subprocess.run([gcc, "-std=c11", "-O1", "-g", "-fPIC", "-shared", "-ffp-contract=off", "-fsanitize=address,undefined",
                    "-fno-sanitize-recover=all", "-o", so, csrc, "-lm"], check=True)
    env = dict(os.environ, LD_PRELOAD=libasan, ASAN_OPTIONS="detect_leaks=0:halt_on_error=1")
    run = subprocess.run([sys.executable, "-c", DRIVER, so, ROOT], capture_output=True, text=True, env=env, timeout=600)
    assert run.returncode != 0 and "AddressSanitizer" in run.stderr
