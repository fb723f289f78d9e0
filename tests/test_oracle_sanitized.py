"""The oracle's C file under AddressSanitizer and UndefinedBehaviorSanitizer.

The device-side memory checker is not available for the CUDA kernels, so the evidence that the CHECKER is
sound has to come from elsewhere: this test compiles oracle/decoder.c with -fsanitize=address,undefined
and runs the calls the parity tests rely on (full and cached forward of all three block families, both
dtypes, ragged chunking, rollback and re-feed, long attention rows) in a child process with the
sanitizer runtime preloaded.  Any out-of-bounds access, use of uninitialised stack, signed overflow or
misaligned access in the oracle aborts the child."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent('''
    import ctypes, os, sys
    import numpy as np
    sys.path.insert(0, os.environ["SSD_ROOT"])
    from oracle import decoder as od
    from paper_2311_04951_b200 import synth
    od._OUT = os.environ["SSD_SAN_LIB"]           # the sanitized build instead of the ordinary one
    od._lib = None
    od.build = lambda force=False: od._OUT
    od.set_threads(2)
    archs = [synth.gpt2_like(2, 64, 4, 128, 97, 48), synth.neox_like(2, 64, 2, 128, 130),
             synth.llama_like(2, 128, 1, 192, 131), synth.neox_like(1, 80, 1, 96, 64, dtype=synth.DT_F32),
             synth.neox_like(2, 64, 2, 128, 130).replace(rotary_dim=16)]
    for k, arch in enumerate(archs):
        ws = synth.gen_weights(arch, 10 + k)
        m = od.Model(arch, ws)
        toks = synth.gen_prompt(20 + k, 1, 23, arch.vocab)[0]
        full = m.forward_full(toks)
        c = m.new_cache(40)
        a = c.feed(toks[:7]); b = c.feed(toks[7:8]); d = c.feed(toks[8:23])
        got = np.concatenate([a, b, d])
        assert np.abs(got - full).max() < 1e-4, (k, np.abs(got - full).max())
        c.rollback(11)
        e = c.feed(toks[11:23])
        assert np.abs(e - full[11:]).max() < 1e-4
        try:
            c.feed(np.zeros(40, np.int32))        # does not fit: refused, nothing written
            raise SystemExit("rows that do not fit were accepted")
        except ValueError:
            pass
    kvl = synth.gen_kv_fill(3, (2, 2, 300, 64), 0)
    q = synth.gen_logits(4, 5, 128)
    od.attention_rows(q, kvl, 290, 5)
    print("sanitized oracle ok")
''')


def test_oracle_runs_clean_under_asan_and_ubsan(tmp_path):
    lib = str(tmp_path / "liboracle_san.so")
    src = os.path.join(ROOT, "oracle", "decoder.c")
    subprocess.check_call(["gcc", "-O1", "-g", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-fsanitize=address,undefined",
                           "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer", "-o", lib, src, "-lm"])
    asan = subprocess.check_output(["gcc", "-print-file-name=libasan.so"], text=True).strip()
    ubsan = subprocess.check_output(["gcc", "-print-file-name=libubsan.so"], text=True).strip()
    assert os.path.exists(asan) and os.path.exists(ubsan)
    env = dict(os.environ, LD_PRELOAD=f"{asan} {ubsan}", SSD_ROOT=ROOT, SSD_SAN_LIB=lib,
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=1", UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    out = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, env=env, timeout=600)
    assert out.returncode == 0, (out.stdout[-1500:], out.stderr[-3000:])
    assert "sanitized oracle ok" in out.stdout
