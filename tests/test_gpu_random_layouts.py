"""Parity on seeded random layouts: head dim, GQA ratio, kept-dim counts, period, residue classes, number
of coefficients, window sizes, prompt length, storage dtype, decode algorithm, reconstruction weights,
frequency grid of the inputs and query sharpness are all drawn at random; every drawn case checks the cache
after compression, a decode call, up to three steps (fused, or append + decode) and the cache again against
the oracle.  Layouts the requested algorithm cannot serve are skipped inside the draw.  One seed draws layouts
with more (batch row, KV head) pairs than the GPU has SMs (8 to 32 KV heads, batch 3 to 11).

Output tolerance: the stated absolute one times max(1, largest |expected output|).  With the paper-literal
weights (1/k instead of 2/T) the compressed part of the outputs is scaled by T / 2k, up to 512 here, and an
absolute bound below the bf16 rounding of such values would test nothing."""
import random

import numpy as np
import pytest

from paper_2506_11886_b200 import fa, synth
from tests.parity_util import OUT_ABS_BF16, OUT_ABS_F32, make_pair

pytestmark = pytest.mark.gpu


def _draw(rng, many_heads=False):
    d = rng.choice([64, 128])
    if many_heads:    # up to 352 (batch row, KV head) pairs for 148 SMs: lone CTAs in waves, two to an SM for short transforms
        Hkv, G, B = rng.choice([8, 16, 32]), rng.choice([1, 2, 4]), rng.choice([3, 5, 8, 11])
    else:
        Hkv, G, B = rng.choice([1, 2, 4]), rng.choice([1, 2, 3, 4, 8]), rng.choice([1, 1, 2, 3])
    nfk, nfv = (min(rng.choice([0, 8, 16, 24, 32, 48, 64]), d) for _ in range(2))
    T = 1 << (rng.choice([8, 9, 10, 11]) if many_heads else rng.choice([8, 9, 10, 11, 12]))
    P = rng.choice([1, 2, 4, 8, 16, 32])
    if T // P < 32:
        return None
    k = min(rng.choice([4, 8, 16, 32, 64, 128, 256]), T // P, T // 2)
    l_init, l_local = rng.choice([0, 1, 4, 7]), rng.choice([0, 5, 16, 64, 100])
    L = rng.randint(0, min(T + l_init + l_local, 1200 if many_heads else 3000))
    algo = rng.choice([fa.FA_DECODE_AUTO, fa.FA_DECODE_FFT, fa.FA_DECODE_FFT if many_heads else fa.FA_DECODE_FFT_SPLIT])
    norm, freq = rng.choice([fa.FA_NORM_ORTHO, fa.FA_NORM_ORTHO, fa.FA_NORM_PAPER]), rng.choice(["grid", "offgrid"])
    shape = synth.Shape("random", B=B, layers=1, Hq=Hkv * G, Hkv=Hkv, d=d, L=L, dtype="bf16" if many_heads else rng.choice(["bf16", "bf16", "f32"]),
                        n_full_k=nfk, n_full_v=nfv, M=2 * k, T=T, L_init=l_init, L_local=l_local, decode_steps=3)
    return shape, P, algo, norm, freq


@pytest.mark.parametrize("seed,many_heads", [(1, False), (2, False), (3, False), (4, True)])
def test_random_layouts(seed, many_heads):
    rng = random.Random(seed)
    done = 0
    for trial in range(14 if many_heads else 40):
        drawn = _draw(rng, many_heads)
        if drawn is None:
            continue
        shape, P, algo, norm, freq = drawn
        try:
            pair, stream = make_pair(shape, seed=1000 * seed + trial, algo=algo, P=P, max_mid=shape.T, norm=norm, freq=freq)
        except fa.FaError as e:
            if e.status in (fa.FA_ERR_UNSUPPORTED, fa.FA_ERR_CAPACITY):
                continue
            raise
        what = f"seed {seed} trial {trial}: {shape} P={P} algo={algo} norm={norm} freq={freq}"
        base = OUT_ABS_F32 if shape.dtype == "f32" else OUT_ABS_BF16

        def close(got, want):
            # the stated absolute tolerance with the orthogonal weights; with the literal 1/k scale the
            # compressed part of the outputs is multiplied by T / 2k, so the bound follows the output magnitude
            bound = base * max(1.0, float(np.abs(want).max())) if norm == fa.FA_NORM_PAPER else base
            err = np.abs(got - want).max()
            assert err <= bound, f"output error {err:.3e} > {bound:.3e}"

        try:
            pair.check_state()
            close(*pair.decode(synth.queries(shape, seed=trial)))
            steps = min(3, shape.T - max(0, shape.L - shape.L_init - shape.L_local))
            K, V = stream.tokens(shape.L, shape.L + max(steps, 1))
            for t in range(steps):
                # (sharpened queries only with the orthogonal weights: the literal scale already multiplies the
                # compressed scores by T / 2k, and a softmax that sharp amplifies rounding beyond any fixed bound)
                peak = rng.choice([1.0, 6.0]) if norm == fa.FA_NORM_ORTHO else 1.0
                q = synth.queries(shape, seed=trial, step=t + 1, peak=peak)
                if rng.random() < 0.5:
                    close(*pair.step(q, K[:, t], V[:, t]))
                else:
                    pair.append(K[:, t], V[:, t])
                    close(*pair.decode(q))
            pair.check_state()
        except AssertionError as e:
            raise AssertionError(f"{what}: {e}") from e
        done += 1
    assert done >= (8 if many_heads else 15)
