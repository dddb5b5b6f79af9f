"""Pins of the oracle's raw-variate gather (Sec. 3.3: the dropped variates leave the lookback window before the embedding):
it is numpy's index-select on the variate axis, and it composes with the selection the way the paper's delta says."""
import numpy as np

import oracle


def test_gather_rows_is_index_select_on_the_variate_axis():
    rng = np.random.default_rng(3)
    x = rng.normal(size=(3, 17, 10)).astype(np.float32)
    sel = np.full((1, 17), -1, np.int32)
    kept = np.array([0, 3, 4, 9, 16], np.int32)
    sel[0, :5] = kept
    out = oracle.gather_rows(x, sel, np.array([5], np.int32), fill=7.0)
    assert np.array_equal(out[:, :5], x[:, kept])            # the library special case: fancy indexing
    assert np.all(out[:, 5:] == 7.0)                         # nothing else is written


def test_gather_rows_per_instance_selection_and_identity():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(4, 9, 6)).astype(np.float32)
    sel = np.full((4, 9), -1, np.int32)
    n_sel = np.array([9, 1, 4, 0], np.int32)
    picks = [np.arange(9), np.array([8]), np.array([1, 2, 5, 7]), np.array([], int)]
    for b, p in enumerate(picks):
        sel[b, : len(p)] = p
    out = oracle.gather_rows(x, sel, n_sel, fill=-1.0)
    assert np.array_equal(out[0], x[0])                      # keeping everything in order is the identity
    for b, p in enumerate(picks):
        assert np.array_equal(out[b, : len(p)], x[b, p]) and np.all(out[b, len(p):] == -1.0)


def test_gather_rows_keeps_one_member_per_group_at_gs_1():
    # with gs = 1 every group keeps exactly one variate (Eq. 1), so the gathered window has one row per distinct hash and
    # hashing the gathered rows again gives pairwise distinct keys
    from paper_2501_14183_b200 import inputs
    w = inputs.WORKLOADS["tiny"]
    x = inputs.make_windows(w)
    keys, _, _ = oracle.hash(x, w.k)
    s = oracle.select(keys, 1, 1.0, 5, 0)
    n = int(s["n_sel"][0])
    assert n == int(s["n_groups"][0])
    xs = oracle.gather_rows(x, s["sel_idx"], s["n_sel"])
    again, _, _ = oracle.hash(xs[:, :n], w.k)
    assert len(set(again[0].tolist())) == n
    assert set(again[0].tolist()) == set(keys[0].tolist())
