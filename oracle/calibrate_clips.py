"""Bisect the noise level s0 of the anchored-scene clip family so that the CPU oracle removes a target
fraction of the tokens at t = 0.70 (about two thirds, the redundancy the paper reports on real video, Table 1).

Run once; the values it prints are frozen in paper_2605_07355_b200/clips.py (_S0).  It calls only the oracle
and the clip generators:   python -m oracle.calibrate_clips [name ...]
"""
from __future__ import annotations

import sys
from dataclasses import replace

from oracle import ttf_oracle as O
from paper_2605_07355_b200 import clips

TARGET = {"tiny": 0.50, "vl2b": 0.67, "vl8b": 0.67, "long": 0.67, "wide": 0.67}
CLIPS_USED = {"long": 3}          # clips of the batch used while bisecting (the check at the end uses all)


def rho_of(spec, s0: float, nclips: int) -> float:
    cal = clips._anchored(spec)
    scale = s0 / cal.sigma
    kw = dict(sigma=s0)
    if cal.sigma_range is not None:
        kw["sigma_range"] = (cal.sigma_range[0] * scale, cal.sigma_range[1] * scale)
    cal = replace(cal, **kw)
    kept = total = 0
    for j in range(nclips):
        X = clips.make_clip(cal, cal.seed + j)
        R = O.compress(X, cal.r, 0.70)
        kept += R.count
        total += R.keep.size
    return 1.0 - kept / total


def main(names):
    for name in names:
        spec = clips.CONFIGS[name]
        n = CLIPS_USED.get(name, spec.clips)
        lo, hi = 0.05, 2.0                      # rho decreases as the noise grows
        for _ in range(12):
            mid = 0.5 * (lo + hi)
            rho = rho_of(spec, mid, n)
            print(f"  {name}: s0={mid:.4f} rho={rho:.4f}", flush=True)
            if rho > TARGET[name]:
                lo = mid
            else:
                hi = mid
            if abs(rho - TARGET[name]) < 0.003:
                break
        print(f"{name}: s0 = {mid:.4f}  rho(0.70) = {rho_of(spec, mid, spec.clips):.4f} over {spec.clips} clip(s)",
              flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or list(TARGET))
