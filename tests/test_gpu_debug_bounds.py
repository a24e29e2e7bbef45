"""The checked build of the library (liblqer_dbg.so, -DLQER_DEBUG_BOUNDS): every global store of the inference
kernels and every copy of packed weights checks its byte range against the extent of its buffer; a violation goes to
the status word and the access is skipped.  It stands in for a memory checker.

The library is process wide, so the checked build runs in child processes (LQER_DEBUG_BOUNDS=1 makes the binding
load it): the small parity cases of the main suite must pass under it with a clean status word, and a launch whose Y is
declared shorter than it is (the build's own test hook) must report LQER_ERR_BOUNDS, leave the bytes beyond the
declared extent untouched and leave the context usable.
"""
import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, timeout=900):
    env = dict(os.environ, LQER_DEBUG_BOUNDS="1")
    return subprocess.run([sys.executable, *args], cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_small_parity_cases_pass_under_the_checked_build():
    # every path of the layer on the small specs: prepare, both prologues, both GEMMs, the decode kernels, shared
    # launches, bf16 and MXINT8 boundaries; each test polls the status word, so a bounds report fails it
    r = _run(["-m", "pytest", "-x", "-q", "-m", "gpu",
              "tests/test_gpu_parity.py", "tests/test_gpu_bf16_io.py", "tests/test_gpu_mxint8_io.py", "tests/test_gpu_w2.py",
              "tests/test_gpu_small_mma.py",
              "-k", "not full and not stack and not sweep and not round"])
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


def test_a_short_extent_is_reported_and_nothing_beyond_it_is_written():
    code = textwrap.dedent("""
        import numpy as np, torch
        import lqer_inputs as gen
        import paper_2402_02446_b200 as L
        from paper_2402_02446_b200 import binding
        assert binding.DEBUG_BOUNDS and L.lib_path().endswith("liblqer_dbg.so")
        E = binding.STATUS_NAMES.index
        dev = "cuda:0"
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        for M, path in ((3, binding.PATH_AUTO), (9, binding.PATH_SMALL), (40, binding.PATH_AUTO), (300, binding.PATH_AUTO)):
            spec = gen.LayerSpec("short", M=M, K=512, N=384, k=16, calib_rows=32, outlier_frac=0.01, outlier_scale=20.0, seed=501)
            W = gen.make_weight(spec); A, B = gen.make_random_factors(spec)
            Pg = L.prepare_weights(t(W), t(A), t(B))
            X = t(gen.make_activations(spec))
            ws = L.new_workspace(M, Pg)
            L.set_path(path)
            Y_good = L.linear(X, Pg, ws).clone()
            assert L.poll_status(ws) == 0
            cut = 4 * 100                                   # the last hundred floats of Y are declared out of range
            Y = torch.full((M, spec.N), 7.0, dtype=torch.float32, device=dev)
            L.debug_bounds_shrink(cut)
            try:
                L.linear(X, Pg, ws, Y)
                torch.cuda.synchronize()
            finally:
                L.debug_bounds_shrink(0)
            assert L.poll_status(ws) == E("LQER_ERR_BOUNDS"), (M, L.poll_status(ws))
            flat, good = Y.flatten(), Y_good.flatten()
            assert torch.all(flat[-100:] == 7.0)            # the guarded stores were skipped
            assert torch.equal(flat[:-128], good[:-128])    # everything clear of the cut was written as usual
            assert L.lib().lqer_workspace_init(ws.data_ptr(), ws.numel(), None) == 0
            assert torch.equal(L.linear(X, Pg, ws), Y_good) and L.poll_status(ws) == 0
            L.set_path(binding.PATH_AUTO)
            Pg.release()
        print("checked-build-ok")
    """)
    r = _run(["-c", code])
    assert r.returncode == 0 and "checked-build-ok" in r.stdout, r.stdout[-3000:] + r.stderr[-3000:]


def test_the_ordinary_build_has_no_such_hook():
    import paper_2402_02446_b200 as L
    from paper_2402_02446_b200 import binding
    if binding.DEBUG_BOUNDS:
        pytest.skip("this process runs the checked build")
    assert L.lib().lqer_debug_bounds_shrink(16) == binding.STATUS_NAMES.index("LQER_ERR_CONFIG")
