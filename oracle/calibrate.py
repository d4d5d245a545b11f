"""TEST INFRASTRUCTURE -- writes ``workloads/params/<config>.json``.

Runs the oracle's calibration (``oracle.networks.calibrate``) on image 0 of each
full-size benchmark configuration and stores every layer's integer parameters, so that
benchmarks and full-size parity tests need not repeat it.  Doubles are stored as
``float.hex`` strings.  Usage: ``python -m oracle.calibrate [config ...]``.
"""
import json
import os
import sys
import time

from workloads import networks as N

from . import networks as ON

OUT_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "workloads", "params")
CONFIGS = ("single_conv", "vdsr", "vrcnn", "resnet18", "resnet50", "resnet152")


def write(name: str) -> str:
    net = N.by_name(name)
    t0 = time.time()
    params = ON.calibrate(net)
    layers = {}
    for k, p in params.items():
        q = dict(p)
        for key in ("delta",):
            if key in q:
                q[key] = float(q[key]).hex()
        layers[k] = q
    t = net.tensors[net.input]
    doc = dict(config=name, seed=net.seed, calibration_image=0, input=[t.h, t.w, t.c],
               written_by="python -m oracle.calibrate", layers=layers)
    path = os.path.join(OUT_DIR, name + ".json")
    with open(path, "w") as f:
        json.dump(doc, f, indent=1, sort_keys=True)
    print("%s: %d layers, %.1f s -> %s" % (name, len(layers), time.time() - t0, path))
    return path


if __name__ == "__main__":
    os.makedirs(OUT_DIR, exist_ok=True)
    for name in (sys.argv[1:] or CONFIGS):
        write(name)
