"""Pins for the oracle's temperature sampler (Gumbel-max with a counter-based generator), CPU only."""
import math

import numpy as np

from paper_2504_12329_b200 import workloads as W

MASK = (1 << 64) - 1


def _sm64_nth(s, n):   # SplitMix64 (Steele, Lea, Flood 2014) in Python integers
    z = (s + n * 0x9E3779B97F4A7C15) & MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK
    return z ^ (z >> 31)


def test_gumbel_variates_follow_their_definition(oracle):
    for seed, step, i in [(0, 0, 0), (7, 3, 151935), (1 << 40, 65000, 12), (MASK, 2**32 - 1, 2**32 - 1)]:
        x = _sm64_nth(seed, ((step << 32) | i) + 1)
        u = ((x >> 41) + 0.5) / 2**23
        assert 0.0 < u < 1.0
        assert oracle.gumbel(seed, step, i) == -math.log(-math.log(u))
    # a standard Gumbel sample: mean = Euler's constant, variance = pi^2 / 6
    g = np.array([oracle.gumbel(11, 5, i) for i in range(200_000)])
    assert abs(g.mean() - 0.5772156649) < 0.01 and abs(g.var() - math.pi**2 / 6) < 0.03


def test_sampled_frequencies_are_the_softmax(oracle):
    """Closed form on a 4-token distribution: argmax of logit / T + Gumbel noise is softmax(logits / T) distributed."""
    z = np.array([1.0, 0.0, -1.0, 2.5])
    for T in (0.7, 1.0, 2.0):
        p = np.exp(z / T) / np.exp(z / T).sum()
        n = 40_000
        counts = np.bincount([oracle.sample(z, T, 123, step)[0] for step in range(n)], minlength=4)
        chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
        assert chi2 < 21.1, (T, counts, n * p)          # 3 degrees of freedom: p < 1e-4
    # the same counter gives the same token; the margin is the gap of the perturbed values
    a, m = oracle.sample(z, 1.0, 5, 9)
    assert (a, m) == oracle.sample(z, 1.0, 5, 9) and m > 0


def test_zero_temperature_and_ties(oracle):
    rng = np.random.default_rng(0)
    z = rng.standard_normal(5000)
    assert oracle.sample(z, 0.0, 1, 2) == oracle.argmax(z)
    for step in range(50):   # a very low temperature is greedy whenever the greedy margin dwarfs T * noise
        assert oracle.sample(z, 1e-4, 1, step)[0] == int(np.argmax(z))
    # only ids below the limit compete
    z2 = np.array([0.0, 0.0, 0.0, 100.0])
    assert oracle.sample(z2, 1.0, 1, 0, limit=3)[0] in (0, 1, 2)


def test_generation_with_sampling(oracle):
    cfg_s = oracle.Config(**W.TINY_S.as_dict())
    ms = oracle.Model(cfg_s, 0, 0)
    prompt = W.prompt_ids(3, 8, 1024)
    kw = dict(delimiter_id=10, keyword_ids=[], n1=3, max_new_tokens=24)
    greedy = oracle.generate_spec(ms, None, prompt, **kw)
    a = oracle.generate_spec(ms, None, prompt, temperature=1.0, sample_seed=5, **kw)
    b = oracle.generate_spec(ms, None, prompt, temperature=1.0, sample_seed=5, **kw)
    c = oracle.generate_spec(ms, None, prompt, temperature=1.0, sample_seed=6, **kw)
    assert a.tokens.tolist() == b.tokens.tolist() != c.tokens.tolist()
    assert a.tokens.tolist() != greedy.tokens.tolist()
    # the first token by hand: the sampler applied to the logits of the prompt's last position, counter = step 0
    z = oracle.KV(ms, 16).forward(prompt)
    assert a.tokens[0] == oracle.sample(z, 1.0, 5, 0)[0]
    # temperature -> 0 is the greedy stream
    cold = oracle.generate_spec(ms, None, prompt, temperature=1e-5, sample_seed=5, **kw)
    assert cold.tokens.tolist() == greedy.tokens.tolist()


def test_nucleus_closed_form_on_four_tokens(oracle):
    """Top-p on a distribution small enough to do by hand.  With z = ln p the softmax at T = 1 is p itself:
    p = (0.5, 0.25, 0.15, 0.1), cumulative 0.5, 0.75, 0.9, 1.0 in order of probability."""
    p = np.array([0.15, 0.5, 0.1, 0.25])           # ids in no particular order
    z = np.log(p)
    members = lambda top_p, T=1.0: [i for i in range(4) if z[i] >= oracle.nucleus_threshold(z, T, top_p)[0]]
    assert members(0.3) == [1]                      # the most probable id alone already holds 0.5 >= 0.3
    assert members(0.5) == [1]                      # "at least top_p": 0.5 reaches 0.5
    assert members(0.6) == [1, 3]                   # 0.5 < 0.6 <= 0.75
    assert members(0.76) == [0, 1, 3]
    assert members(0.95) == [0, 1, 2, 3]
    # the reported gap is the distance of top_p to the nearer cumulative sum around the cut
    assert abs(oracle.nucleus_threshold(z, 1.0, 0.6)[1] - 0.1) < 1e-12
    assert abs(oracle.nucleus_threshold(z, 1.0, 0.74)[1] - 0.01) < 1e-12
    # the temperature acts before the cut: at T = 0.5 the probabilities are p^2 / sum = (.0625, .25, .0225, .01) / .345
    assert members(0.7, T=0.5) == [1]               # 0.7246 >= 0.7
    assert members(0.8, T=0.5) == [1, 3]            # 0.7246 < 0.8 <= 0.9058
    # ids that tie with the last member come along, whatever their order
    zt = np.log(np.array([0.2, 0.4, 0.2, 0.2]))
    assert [i for i in range(4) if zt[i] >= oracle.nucleus_threshold(zt, 1.0, 0.5)[0]] == [0, 1, 2, 3]
    # only ids below the limit count
    z5 = np.append(z, 10.0)
    assert oracle.nucleus_threshold(z5, 1.0, 0.6, limit=4)[0] == oracle.nucleus_threshold(z, 1.0, 0.6)[0]


def test_top_p_sampling_is_the_renormalised_distribution(oracle):
    p = np.array([0.15, 0.5, 0.1, 0.25])
    z = np.log(p)
    # nucleus {1, 3} renormalised: (2/3, 1/3); nothing else is ever drawn
    n = 30_000
    draws = [oracle.sample_top_p(z, 1.0, 0.6, 77, step)[0] for step in range(n)]
    counts = np.bincount(draws, minlength=4)
    assert counts[0] == 0 and counts[2] == 0
    want = n * np.array([2 / 3, 1 / 3])
    chi2 = float(((counts[[1, 3]] - want) ** 2 / want).sum())
    assert chi2 < 15.1, counts                       # 1 degree of freedom: p < 1e-4
    # top_p outside (0, 1) is no restriction: the same draws as plain temperature sampling
    for step in range(200):
        assert oracle.sample_top_p(z, 1.0, 1.0, 9, step)[0] == oracle.sample(z, 1.0, 9, step)[0]
        assert oracle.sample_top_p(z, 1.0, 0.0, 9, step)[0] == oracle.sample(z, 1.0, 9, step)[0]
    # a nucleus of one id is greedy
    rng = np.random.default_rng(1)
    big = rng.standard_normal(3000)
    for step in range(50):
        assert oracle.sample_top_p(big, 1.0, 1e-6, 3, step)[0] == int(np.argmax(big))
    # inside the nucleus the draw is the unrestricted Gumbel-max draw whenever that one falls inside
    thr, _ = oracle.nucleus_threshold(big, 1.0, 0.9)
    same = 0
    for step in range(300):
        free = oracle.sample(big, 1.0, 4, step)[0]
        if big[free] >= thr:
            assert oracle.sample_top_p(big, 1.0, 0.9, 4, step)[0] == free
            same += 1
    assert same > 200


def test_generation_with_top_p(oracle):
    cfg_s = oracle.Config(**W.TINY_S.as_dict())
    ms = oracle.Model(cfg_s, 0, 0)
    prompt = W.prompt_ids(3, 8, 1024)
    kw = dict(delimiter_id=10, keyword_ids=[], n1=3, max_new_tokens=24, temperature=1.0, sample_seed=5)
    free = oracle.generate_spec(ms, None, prompt, **kw)
    cut = oracle.generate_spec(ms, None, prompt, top_p=0.5, **kw)
    assert cut.tokens.tolist() != free.tokens.tolist()
    z = oracle.KV(ms, 16).forward(prompt)
    assert cut.tokens[0] == oracle.sample_top_p(z, 1.0, 0.5, 5, 0)[0]
    assert oracle.generate_spec(ms, None, prompt, top_p=1.0, **kw).tokens.tolist() == free.tokens.tolist()
