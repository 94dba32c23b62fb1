"""Test infrastructure: the paper's accounting written out term by term (appendix "Computation of FLOPs", Eq.
"Estimated Speed", the modify ratio of the results tables), with plain loops.  Only tests may import this."""


def flops_prefill(s, h, hp, n):
    return 8 * s * h ** 2 + 16 * s * h + 4 * s ** 2 * h + 4 * s ** 2 * n + 6 * s * h * hp + 2 * s * hp


def flops_decode(s, h, hp, n):
    return 8 * h ** 2 + 16 * h + 4 * s * h + 4 * s * n + 6 * h * hp + 2 * hp


def flops_total(prompt_len, n_new, h, hp, n):
    total = flops_prefill(prompt_len, h, hp, n)
    for i in range(n_new):
        total += flops_decode(prompt_len + i, h, hp, n)
    return total


def estimated_speed_plain(prompt_len, n_new, h, hp, n, capacity=3.12e10):
    return n_new / (flops_total(prompt_len, n_new, h, hp, n) / capacity)


def modify_ratio(source):
    return sum(1 for s in source if s == 1) / max(1, len(source))
