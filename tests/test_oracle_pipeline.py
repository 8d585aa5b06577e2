"""Whole-path pins for the oracle: planted hubs are recovered through the global
centrality while a single-layer snapshot misses dormant ones (the paper's thesis,
Sections 1 and 3.1), the stored micro-workload results, and the generator's
determinism."""
import importlib.util
import os

import numpy as np
import pytest
import torch

from oracle import structkv_oracle as O
from paper_2604_06746_b200 import synth


def oracle_layers(wl, pl):
    out = []
    for l in range(wl.n_layers):
        t = synth.make_layer(wl, pl, l, with_v=False)
        out.append((synth.to_f64(t["q_win"]), synth.to_f64(t["k"]), t["scale"]))
    return out


@pytest.fixture(scope="module")
def tiny_run():
    wl = synth.WORKLOADS["tiny"]
    pl = synth.plan(wl)
    layers = oracle_layers(wl, pl)
    return wl, pl, {w: O.prefill(layers, wl.window, wl.budget, wl.struct_budget(), weights=w)
                    for w in (O.PAPER_WEIGHTS, (1.0, 0.0, 0.0))}


def test_tiny_entropy_pivot_is_unique(tiny_run):
    wl, pl, runs = tiny_run
    r = runs[(1.0, 0.0, 0.0)]
    ent = r["metrics"][:, 0]
    assert ent[0] < ent[1] < ent[2] > ent[3]          # temperatures 0.5, 1, 2, 1
    assert r["pivot"] == 3
    for run in runs.values():
        T = np.sort(run["transition"][1:])[::-1]
        assert T[0] - T[1] >= 0.05


def test_tiny_invariants(tiny_run):
    wl, pl, runs = tiny_run
    r = runs[(1.0, 0.0, 0.0)]
    np.testing.assert_allclose(r["s_hist"].sum(axis=1), wl.n_q_heads, rtol=1e-10)
    lam, p = O.PAPER_LAMBDA, r["pivot"]
    assert abs(r["C"].sum() - wl.n_q_heads * (1 - lam ** (p + 1)) / (1 - lam)) < 1e-9
    assert np.all((r["metrics"][:, 0] >= 0) & (r["metrics"][:, 0] <= np.log(wl.seq)))


def test_tiny_hubs_recovered_by_centrality_not_by_snapshot(tiny_run):
    wl, pl, runs = tiny_run
    r = runs[(1.0, 0.0, 0.0)]
    hubs = set(pl.hub_positions.tolist())
    assert hubs <= set(r["i_struct"].tolist())
    # hubs are dormant at the pivot layer: a snapshot of that layer alone finds few of them
    snap = O.select(r["s_hist"][r["pivot"]], wl.struct_budget(), wl.window)
    assert len(hubs & set(snap.tolist())) <= len(hubs) // 2
    # decoupled KV sets follow the local saliency: all hubs where active, few where dormant
    for l in (1, 2):
        assert hubs <= set(r["i_kv"][l].tolist())
    assert len(hubs & set(r["i_kv"][3].tolist())) <= len(hubs) // 2
    # the sets are independent, each with its own budget
    assert len(r["i_struct"]) == wl.struct_budget() and r["i_kv"].shape == (4, wl.budget)


def test_scaled_workloads_recover_active_hubs():
    for name, seq, hubs in (("llama32k", 2048, 8), ("qwen64k", 2048, 8)):
        wl = synth.WORKLOADS[name].scaled(seq, n_layers=6, n_hubs=hubs, budgets=(256,))
        pl = synth.plan(wl)
        r = O.prefill(oracle_layers(wl, pl), wl.window, wl.budget, wl.struct_budget())
        p = r["pivot"]
        active_near = [int(pos) for h, pos in enumerate(pl.hub_positions)
                       if pl.hub_active[max(0, p - 2):p + 1, h].any()]
        assert set(active_near) <= set(r["i_struct"].tolist()), name


def test_micro_workload_matches_stored_results():
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "golden", "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    s = mg.SHAPE
    r = O.prefill(mg.micro_inputs(), s["w"], s["kv_budget"], s["struct_budget"])
    with open(os.path.join(here, "golden", "micro_prefill.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            tag, *rest = line.split()
            if tag == "pivot":
                assert r["pivot"] == int(rest[0])
            elif tag == "metrics":
                np.testing.assert_allclose(r["metrics"][int(rest[0])], [float(x) for x in rest[1:]], rtol=1e-12)
            elif tag == "C":
                np.testing.assert_allclose(r["C"], [float(x) for x in rest], rtol=1e-12)
            elif tag == "i_struct":
                assert r["i_struct"].tolist() == [int(x) for x in rest]
            elif tag == "i_kv":
                assert r["i_kv"][int(rest[0])].tolist() == [int(x) for x in rest[1:]]


def test_generator_is_deterministic_and_structured():
    wl = synth.WORKLOADS["llama128k"].scaled(4096, n_layers=10, n_hubs=16)
    pl, pl2 = synth.plan(wl), synth.plan(wl)
    assert np.array_equal(pl.hub_positions, pl2.hub_positions) and np.array_equal(pl.hub_active, pl2.hub_active)
    assert len(set(pl.hub_positions.tolist())) == 16
    assert pl.hub_positions.min() >= 1 and pl.hub_positions.max() < wl.seq - wl.window
    assert np.all(pl.hub_active.sum(axis=0) == 8)            # contiguous 8-layer spans
    assert np.all((pl.temperatures >= 0.5) & (pl.temperatures <= 2.0))
    a, b = synth.make_layer(wl, pl, 3), synth.make_layer(wl, pl, 3)
    for key in ("q_win", "k", "v"):
        assert a[key].dtype.is_floating_point and a[key].dtype == synth.torch_dtype(wl.dtype)
        assert (a[key].view(dtype=torch.int16) == b[key].view(dtype=torch.int16)).all()
    k = synth.to_f64(a["k"])
    norms = np.linalg.norm(k[0], axis=1)
    assert norms[0] > 2.5 * np.median(norms)                 # sink
    assert np.median(norms[10::20]) < 0.2 * np.median(norms) # delimiters
    c = synth.make_layer(wl, pl, 4)
    assert not (a["k"].view(dtype=torch.int16) == c["k"].view(dtype=torch.int16)).all()
