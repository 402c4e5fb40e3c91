"""Loaders of the hand-worked text fixtures under tests/golden/ (no arithmetic of the method in here)."""
import os

import numpy as np

GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_spine_tree_example():
    """tests/golden/spine_tree_hand_example.txt -> dict (inputs, the adjacency table as int32 [rows][K], expected trees)."""
    ex = {"cases": [], "rows": {}}
    for line in open(os.path.join(GOLDEN_DIR, "spine_tree_hand_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(None, 1)
        if key == "adj":
            t, ids = rest.split(":")
            ex["rows"][int(t)] = [int(v) for v in ids.split()]
        elif key == "case":
            D, tok, par, ns = [t.strip() for t in rest.split("|")]
            ex["cases"].append((int(D), [int(v) for v in tok.split()], [int(v) for v in par.split()], int(ns)))
        elif key in ("r", "rho"):
            ex[key] = float(rest)
        elif key in ("anchor", "B", "table_rows", "K"):
            ex[key] = int(rest)
        else:
            ex[key] = [int(v) for v in rest.split()]
    adj = np.full((ex["table_rows"], ex["K"]), -1, np.int32)
    for t, ids in ex["rows"].items():
        adj[t, :len(ids)] = ids
    ex["adj"] = adj
    return ex
