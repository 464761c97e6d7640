"""Seeded sweep over randomly drawn shapes, head layouts, tolerances and presets for every entry point, each case
checked against the fp64 oracle by the helpers of the other GPU test files."""
import random

import pytest

from paper_2609_32712_b200 import workloads as W
from tests import test_gpu_bwd as TB
from tests import test_gpu_chunk as TC
from tests import test_gpu_decode as TD
from tests import test_gpu_fwd as TF
from tests import test_gpu_varlen as TV

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mala():
    from paper_2609_32712_b200 import mala as m
    m.lib()
    return m


def _heads(rng):
    hkv, g = rng.choice([1, 2, 3]), rng.choice([1, 2, 4])
    return hkv * g, hkv


@pytest.mark.parametrize("seed", [2, 3, 4])
def test_random_cases(mala, oracle, seed):
    _sweep(mala, oracle, seed, [64, 128], 40)


@pytest.mark.parametrize("seed", [5, 6])
def test_random_cases_any_head_size(mala, oracle, seed):
    _sweep(mala, oracle, seed, list(range(8, 129, 8)), 40)


def _sweep(mala, oracle, seed, head_sizes, n):
    rng = random.Random(seed)
    for it in range(n):
        kind = rng.choice(["fwdbwd", "chunk", "split", "varlen", "decode", "paged", "multi"])
        tau = rng.choice([0.0, 1e-5, 1e-4, 1e-2, 1.0])
        d = rng.choice(head_sizes)
        preset = rng.choice(["literal", "R"])
        if kind == "fwdbwd":
            Hq, Hkv = _heads(rng)
            N, causal = rng.randint(1, 1400), rng.random() < 0.8
            w = W.custom_prefill(rng.choice([1, 2]), Hq, Hkv, N, d, seed=rng.randint(0, 9999), preset=preset)
            TF._run_and_check(mala, oracle, w, tau, causal=causal)
            TB._run_isolated(mala, oracle, w, tau, causal=causal)
        elif kind in ("chunk", "split"):
            Hq, Hkv = _heads(rng)
            Nq, off, causal = rng.randint(1, 700), 128 * rng.randint(0, 8), rng.random() < 0.8
            Nk = Nq + off if causal else rng.randint(1, 1500)
            w = W.custom_prefill(1, Hq, Hkv, max(Nk, Nq), d, seed=rng.randint(0, 9999), preset=preset)
            if causal:
                c = TC._chunk(w, Nq)
            else:
                c = dict(q=w["q"][:, :Nq].contiguous(), k=w["k"][:, :Nk].contiguous(), v=w["v"][:, :Nk].contiguous(),
                         do=w["do"][:, :Nq].contiguous(), scale=w["scale"])
            S = rng.randint(2, 9)
            if kind == "chunk":
                TC._run(mala, oracle, c, tau, causal=causal)
            else:
                TC._run_split(mala, oracle, c, tau, S, causal=causal)
                if causal and Nk > Nq + 1:   # the forward also from a position inside a tile, unsplit and split
                    c2 = TC._chunk(w, Nq + rng.randint(1, min(127, Nk - Nq)))
                    TC._run_fwd_any_offset(mala, oracle, c2, tau, rng.choice([1, S]))
                    if len(head_sizes) > 2:   # (the newer sweep: the backward from that position as well)
                        TC._run_bwd_any_offset(mala, oracle, c2, tau)
        elif kind == "varlen":
            Hq, Hkv = _heads(rng)
            lens = [rng.randint(1, 600) for _ in range(rng.randint(1, 4))]
            TV._run(mala, oracle, lens, Hq, Hkv, d, tau, preset=preset, causal=rng.random() < 0.8)
        elif kind == "decode":
            Hkv, G = rng.choice([1, 2, 3]), rng.choice([1, 2, 3, 4, 5, 8, 16])
            Nk, S = rng.randint(1, 5000), rng.randint(1, 12)
            w = W.custom_decode(rng.choice([1, 2, 3]), Hkv * G, Hkv, Nk, d, S, seed=rng.randint(0, 9999),
                                preset=rng.choice(["literal", "D"]))
            TD._run_and_check(mala, oracle, w, tau, S)
        elif kind == "paged":
            Hkv, G, page = rng.choice([1, 2]), rng.choice([1, 2, 4, 8]), rng.choice([128, 256, 512])
            Nk, S, B = page * rng.randint(1, 12), rng.randint(1, 8), rng.choice([1, 2, 3])
            lens = [rng.randint(0, Nk) for _ in range(B)]
            w = W.custom_decode(B, Hkv * G, Hkv, Nk, d, S, seed=rng.randint(0, 9999), preset=rng.choice(["literal", "D"]))
            TD._run_paged(mala, oracle, w, tau, S, page, lens, seed=it)
        else:
            Hkv, G = rng.choice([1, 2]), rng.choice([1, 2, 4])
            Sq = rng.randint(2, 16 // G)
            Nk, S = rng.randint(Sq, 4000), rng.randint(1, 8)
            w = W.custom_decode(rng.choice([1, 2]), Hkv * G, Hkv, Nk, d, S, seed=rng.randint(0, 9999),
                                preset=rng.choice(["literal", "D"]))
            TD._run_multi(mala, oracle, w, Sq, tau, S, seed=it)
