"""The seeded input generator: reproducible, thread-count independent, shaped as stated."""
import os
import subprocess
import sys

import numpy as np

import graphgen as gg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_mix64_is_a_pure_function_of_its_counter():
    assert gg.mix64(0, 1, 2) == gg.mix64(0, 1, 2)
    vals = {gg.mix64(s, t, i) for s in range(3) for t in range(3) for i in range(50)}
    assert len(vals) == 450


def test_powerlaw_graph_shape():
    n = 4096
    src, dst = gg.powerlaw_graph(n, 40_000, 2.1, None, 0)
    assert abs(len(src) - 40_000) <= 400
    assert src.min() >= 0 and src.max() < n and dst.min() >= 0 and dst.max() < n
    assert (src != dst).all()
    key = dst.astype(np.int64) * n + src
    assert len(np.unique(key)) == len(key)
    deg = np.bincount(dst, minlength=n)
    assert deg.min() >= 1 and deg.max() > 20 * deg.mean()      # heavy tail
    assert (np.diff(dst) < 0).any()                            # COO order is shuffled


def test_generation_does_not_depend_on_thread_count():
    code = ("import graphgen as gg, hashlib;"
            "s,d=gg.powerlaw_graph(2000,20000,2.1,None,3);"
            "x=gg.features_f32(100,7,dist='normal',p0=0,p1=1,seed=3);"
            "r=gg.rmat_graph(10,5000,seed=3);"
            "print(hashlib.sha1(s.tobytes()+d.tobytes()+x.tobytes()+r[0].tobytes()+r[1].tobytes()).hexdigest())")
    out = []
    for threads in ("1", "3"):
        env = dict(os.environ, OMP_NUM_THREADS=threads, PYTHONPATH=ROOT)
        out.append(subprocess.check_output([sys.executable, "-c", code], env=env, cwd=ROOT).strip())
    assert out[0] == out[1]


def test_rmat_skew_and_range():
    src, dst = gg.rmat_graph(12, 60_000, seed=0, relabel=False)
    n = 1 << 12
    assert src.min() >= 0 and src.max() < n and dst.max() < n
    # a = 0.57 concentrates mass on low ids before relabelling
    assert (src < n // 2).mean() > 0.7 and (dst < n // 2).mean() > 0.7
    s2, d2 = gg.rmat_graph(12, 60_000, seed=0, relabel=True)
    assert not np.array_equal(src, s2)
    assert np.array_equal(np.sort(np.bincount(src, minlength=n)), np.sort(np.bincount(s2, minlength=n)))


def test_feature_distributions_and_padding():
    u = gg.features_f32(2000, 10, ld=12, dist="uniform", p0=0.0, p1=1.0, seed=1, pad=-7.0)
    assert (u[:, 10:] == -7.0).all() and u[:, :10].min() >= 0 and u[:, :10].max() < 1
    assert abs(u[:, :10].mean() - 0.5) < 0.02
    g = gg.features_f32(4000, 8, dist="normal", p0=0.0, p1=0.1, seed=1)
    assert abs(g.mean()) < 0.005 and abs(g.std() - 0.1) < 0.005


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -0.3, 65504.0], np.float32)
    bits = gg.to_bf16_bits(x)
    back = gg.bf16_bits_to_f32(bits)
    assert back[0] == 1.0
    assert back[1] == 1.0                      # tie -> even mantissa
    assert back[2] == 1.0 + 2.0 ** -6          # tie -> even mantissa (upwards)
    assert abs(back[3] + 0.3) <= 2.0 ** -9 * 0.5
