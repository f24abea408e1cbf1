"""Pins for the oracle's token filter (Algorithm 1 of the paper)."""
import os

import numpy as np
import pytest

import oracle
from helpers import alg1_python

GOLD = os.path.join(os.path.dirname(__file__), "golden", "filter_alg1_hand.txt")


def _gold_cases():
    out = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, kept, left = line.split("|")
        W, N = map(int, head.split())
        out.append((W, N, [int(x) for x in kept.split()], [int(x) for x in left.split()]))
    return out


@pytest.mark.parametrize("W,N,kept,left", _gold_cases())
def test_hand_simulated_cases(W, N, kept, left):
    k, q, ev = oracle.filter_ids(W, N)
    assert k.tolist() == kept
    assert q.tolist() == left
    assert ev == len(left) // W


@pytest.mark.parametrize("W", [1, 2, 3, 4, 5, 8, 16, 42, 64, 128])
def test_matches_literal_python_slices(W):
    for N in sorted({0, 1, 3 * W - 1, 3 * W, 3 * W + 1, 4 * W, 4 * W + 1, 7 * W + 3, 20 * W + 1}):
        A, Q = alg1_python(W, N)
        k, q, ev = oracle.filter_ids(W, N)
        assert k.tolist() == A and q.tolist() == Q


@pytest.mark.parametrize("W", [2, 3, 7, 16, 42, 128])
def test_invariants(W):
    n_events_prev = 0
    for N in range(1, 12 * W + 2):
        k, q, ev = oracle.filter_ids(W, N)
        # partition of 0..N-1
        assert sorted(k.tolist() + q.tolist()) == list(range(N))
        # events fire exactly when token index t = 3W + jW arrives, each moves W tokens
        expect_events = 0 if N <= 3 * W else (N - 1 - 3 * W) // W + 1
        assert ev == expect_events and len(q) == ev * W
        # length of the full-precision list: 2W < len <= 3W after the first event
        if ev:
            assert 2 * W < len(k) <= 3 * W
        else:
            assert len(k) == N
        # token 0 is never filtered out; kept ids ascending
        assert k[0] == 0 and np.all(np.diff(k) > 0)
        # the newest W..2W tokens are consecutive
        if ev:
            run = 1
            while run < len(k) and k[-run - 1] == k[-run] - 1:
                run += 1
            assert W <= run
        n_events_prev = ev
    assert n_events_prev > 0


def test_reserved_budget_of_the_paper():
    # Sec. 3.1/3.2.3: R = 128 gives W = floor(R/3) = 42 and at most 3W = 126 kept tokens.
    W = 128 // 3
    assert W == 42
    mx = max(len(oracle.filter_ids(W, N)[0]) for N in range(1, 700))
    assert mx == 126


@pytest.mark.parametrize("W", [2, 4, 8, 16, 64, 128, 256])
def test_closed_form_power_of_two(W):
    """For W = 2^L: right after event number c (1-based count), the kept set is, in the steady
    state c >= L+1, {0} U union_k { (c+1-k)W + r : r = 0 mod 2^k, 0 <= r < W }, k = 0..L."""
    L = W.bit_length() - 1
    for c in range(1, L + 6):
        N = 3 * W + (c - 1) * W + 1  # the token that triggered event c has just been appended
        k, q, ev = oracle.filter_ids(W, N)
        assert ev == c
        kept_before_new = set(k.tolist()) - {N - 1}
        if c >= L + 1:
            expect = {0}
            for kk in range(L + 1):
                base = (c + 1 - kk) * W
                expect |= {base + r for r in range(0, W, 2 ** kk)}
            assert kept_before_new == expect
        else:
            expect = set(range((c + 1) * W, (c + 2) * W))
            for i in range(2, c + 1):
                expect |= {i * W + r for r in range(0, W, 2 ** (c + 1 - i))}
            expect |= {p for p in range(0, 2 * W, 2 ** c)}
            assert kept_before_new == expect


def test_log_spacing_of_kept_tokens():
    # Sec. 2.2/2.5: density halves window by window going back from the newest tokens.
    W = 64
    k, _, _ = oracle.filter_ids(W, 40 * W + 1)
    newest = k[-1]
    dist = newest - k[:-1]
    for j in range(1, 6):
        lo, hi = j * W, (j + 1) * W  # the window j windows back from the newest token
        cnt = int(np.sum((dist > lo) & (dist <= hi)))
        assert cnt == W // 2 ** j
