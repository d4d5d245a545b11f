"""Cached per-layer parameters of the full-size configurations (``*.json`` beside this file,
written by ``python -m oracle.calibrate``).  A plain JSON reader: none of the method's arithmetic."""
import json
import os

PARAMS_DIR = os.path.dirname(os.path.abspath(__file__))


def load_params(name: str) -> dict:
    """Per-layer parameters of a configuration (``float.hex`` strings for doubles so that the
    quantisation steps round-trip exactly)."""
    name = {"vrcnn_hd": "vrcnn", "vdsr_hd": "vdsr"}.get(name, name)   # the single-picture workloads run the layers of configurations 3 and 2
    with open(os.path.join(PARAMS_DIR, name + ".json")) as f:
        raw = json.load(f)
    for p in raw["layers"].values():
        if "delta" in p:
            p["delta"] = float.fromhex(p["delta"])
    return raw["layers"]
