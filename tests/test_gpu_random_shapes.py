"""Seeded random problem shapes through gc_build_cache against the CPU oracle, element by element:
sizes drawn so that every plan is met (one-tile batches in bf16 and fp32, narrow and wide bf16
rows with ragged tiles and split ranges, the four-CTA sweeps, fp32 batches of a few tiles, the
FMA-tile plan for widths that are not a multiple of 8), both mask modes, several temperatures.
The shapes are fixed by the seed: the same forty-odd cases every run."""
import numpy as np
import pytest
import torch

from paper_2101_06983_b200 import inputs

from gpu_util import check_against_oracle, run_build

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20210106)
    out = []
    widths = {
        "one-tile": [8, 24, 64, 72, 128, 200, 320, 512, 768, 1024],
        "narrow": [64, 128, 192, 256],
        "wide": [320, 384, 448, 576, 1024, 1536],
        "quad": [512, 640, 768],
        "fma": [4, 12, 40, 100, 136, 264],
    }
    for kind, n_cases in (("one-tile", 12), ("narrow", 8), ("wide", 6), ("quad", 6), ("fma", 8)):
        for _ in range(n_cases):
            d = int(rng.choice(widths[kind]))
            if kind == "one-tile":
                dtype = "bf16" if rng.random() < 0.5 else "f32"
                B = int(rng.integers(1, 129))
                N = int(rng.integers(1, 257 if dtype == "bf16" else 129))
            elif kind == "fma":
                dtype = "f32"
                B, N = int(rng.integers(129, 400)), int(rng.integers(129, 500))
            else:
                dtype = "bf16"
                B, N = int(rng.integers(129, 700)), int(rng.integers(257, 1400))
            mask = int(rng.random() < 0.3 and N >= 2)
            tau = float(rng.choice([0.05, 0.2, 0.5, 1.0]))
            out.append((kind, dtype, B, N, d, mask, tau, int(rng.integers(1, 1 << 30))))
    return out


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2101_06983_b200 import binding as b
    return b


@pytest.mark.parametrize("kind,dtype,B,N,d,mask,tau,seed", _cases())
def test_random_shape(binding, oracle, kind, dtype, B, N, d, mask, tau, seed):
    if dtype == "bf16" and d % 8:
        d = (d + 7) // 8 * 8
    if mask:
        n = min(B, N)           # the masked pair is (i, i): keep a positive off the diagonal
        prob = inputs.random_problem(n, n, d, dtype, seed=seed, tau=tau, scale=d ** -0.5,
                                     mask_mode=inputs.MASK_SELF, shared=True)
    else:
        prob = inputs.random_problem(B, N, d, dtype, seed=seed, tau=tau, scale=d ** -0.5)
    code = binding.GC_BF16 if dtype == "bf16" else binding.GC_F32
    plan = binding.gc_plan_name(binding.GC_OP_BUILD, prob.B, prob.N, prob.d, code)
    if kind == "one-tile":
        assert plan == "tcgen05-one-tile"
    if kind == "fma":            # fp32 beyond one tile: tcgen05 per tile pair, or FMA tiles
        assert plan == ("tcgen05-tiles" if prob.d % 8 == 0 else "simt")
    out = run_build(prob)
    ref = oracle.build_cache(prob.Q, prob.P, prob.pos_idx, prob.tau, prob.mask_mode)
    check_against_oracle(prob, out, ref)
