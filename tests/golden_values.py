"""Readers for the fixtures under tests/golden (values the paper prints; not a test module)."""
import json
import os

HERE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def figures():
    with open(os.path.join(HERE, "printed_figures.json")) as f:
        return {k: v["value"] for k, v in json.load(f).items()}


def panel():
    """Table E.2 as {arm: (class, phi, gamma)}."""
    out = {}
    with open(os.path.join(HERE, "table_e2_panel.tsv")) as f:
        for line in f:
            if line.startswith("#") or line.startswith("arm\t") or not line.strip():
                continue
            arm, cls, phi, gamma = line.rstrip("\n").split("\t")
            out[arm] = (cls, float(phi), float(gamma))
    return out
