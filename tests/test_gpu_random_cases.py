"""Seeded random cases: sizes, learner counts, compression rates, value distributions (continuous, heavily
quantised, mostly zero), selectors, layerings, alignment and options drawn at random, three steps each, every
output compared with the oracle element by element.  Meant to reach paths the hand-written cases do not."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _parity():
    from tests import parity
    return parity


def _draw_case(rng):
    d = int(np.exp(rng.uniform(np.log(1), np.log(2_000_000))))
    n = int(rng.integers(1, 10))
    k = int(np.clip(np.exp(rng.uniform(0, np.log(d + 1))), 1, d))
    kind = rng.choice(["normal", "quantised", "sparse", "mixed_scale"])
    steps = 3

    def vec():
        x = rng.standard_normal(d)
        if kind == "quantised":
            x = np.round(x * 2) / 2                      # a dozen distinct magnitudes: ties everywhere
        elif kind == "sparse":
            x = np.where(rng.random(d) < 0.9, 0.0, x)
        elif kind == "mixed_scale":
            x = x * np.exp(rng.uniform(-6, 6))
        return x.astype(np.float32)

    grads = [[vec() for _ in range(n)] for _ in range(steps)]
    selector = rng.choice(["topk", "topk", "chunk", "layer_topk", "chunk_layers"])
    layers = None
    if selector in ("layer_topk", "chunk_layers"):
        nl = int(rng.integers(1, min(d, 12) + 1))
        cuts = np.sort(rng.choice(np.arange(1, d), size=nl - 1, replace=False)) if nl > 1 else np.array([], int)
        sizes = np.diff(np.concatenate([[0], cuts, [d]])).astype(int).tolist()
        keep = [int(rng.integers(1, s + 1)) if rng.random() < 0.7 else s for s in sizes]
        layers = (sizes, keep)
        k = sum(keep)
    return dict(d=d, n=n, k=k, grads=grads, selector="chunk" if selector == "chunk_layers" else selector, layers=layers,
                force_exact=bool(rng.random() < 0.3), fuse_update=bool(rng.random() < 0.7), offset=int(rng.integers(0, 4)),
                use_hint=bool(rng.random() < 0.8), beta=float(rng.choice([0.1, 0.5, 1.0])), t0=int(rng.integers(0, 20)),
                kind=kind)


@pytest.mark.parametrize("seed", range(24))
def test_random_cases_match_the_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    p = _parity()
    for case_no in range(10):
        c = _draw_case(rng)
        tag = "seed %d case %d: d=%d n=%d k=%d %s %s layers=%s exact=%s fuse=%s off=%d hint=%s" % (
            seed, case_no, c["d"], c["n"], c["k"], c["kind"], c["selector"],
            None if c["layers"] is None else len(c["layers"][0]), c["force_exact"], c["fuse_update"], c["offset"], c["use_hint"])
        grads = [[torch.from_numpy(g).to(DEV) for g in step] for step in c["grads"]]
        m0 = [torch.zeros(c["d"], device=DEV) for _ in range(c["n"])]
        theta0 = torch.linspace(-1, 1, c["d"], device=DEV)
        p.run_and_compare(grads, m0, theta0, c["k"], c["beta"], 0.25, t0=c["t0"], force_exact=c["force_exact"],
                          fuse_update=c["fuse_update"], offset=c["offset"], use_hint=c["use_hint"],
                          selector=c["selector"], layers=c["layers"], tag=tag,
                          l2_keep=(c["d"] + c["n"] + c["k"]) % 3 != 0)      # (derived, so that the drawn cases stay the same)
