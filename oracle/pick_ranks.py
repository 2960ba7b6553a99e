"""Writes asi_inputs/energy_ranks.py: per-mode ranks at a given explained-variance
threshold (the HOSVD_eps rule of Sec. 3.2) for the energy-picked benchmark
configurations, computed by the fp64 oracle on each layer's step-0 tensor.

Run from the repository root:  python -m oracle.pick_ranks
Calls only oracle/ and the input generator.
"""
from __future__ import annotations

import os
import sys
import time

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from asi_inputs.configs import CONFIG_CLIP, layer_seed, untuned_layers  # noqa: E402
from asi_inputs.generator import LayerStream  # noqa: E402
from oracle.asi_oracle import mode_spectrum  # noqa: E402

ENERGIES = {1: (0.8, 0.9, 0.95), 2: (0.8, 0.9), 3: (0.8, 0.9, 0.95)}


def main():
    lines = ['"""Energy-picked ranks: (config index, layer index, energy) -> ranks per mode.',
             "",
             "Written by oracle/pick_ranks.py (fp64 eigenvalues of A_m A_m^T on the step-0",
             'tensor of each layer stream).  Do not edit by hand."""',
             "ENERGY_RANKS = {"]
    for ci in (1, 2, 3):
        for li, L in enumerate(untuned_layers(ci)):
            t0 = time.time()
            st = LayerStream(dims=L.dims, ranks=(1,) * len(L.dims), dy_shape=(1, 1, 1, 1),
                             seed=layer_seed(ci, li), clip=CONFIG_CLIP[ci])
            A, _ = st.next()
            A = A.astype(np.float64)
            spectra = [mode_spectrum(A, m) for m in range(A.ndim)]
            for e in ENERGIES[ci]:
                ranks = []
                for m, lam in enumerate(spectra):
                    frac = np.cumsum(lam) / np.sum(lam)
                    r = int(np.searchsorted(frac, e - 1e-15) + 1)
                    ranks.append(max(1, min(r, 64, A.shape[m], A.size // A.shape[m])))
                lines.append(f"    ({ci}, {li}, {e}): {tuple(ranks)},   # {L.name} {L.dims}")
            print(ci, li, L.name, f"{time.time() - t0:.1f}s", flush=True)
    lines.append("}")
    out = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                       "asi_inputs", "energy_ranks.py")
    with open(out, "w") as f:
        f.write("\n".join(lines) + "\n")
    print("wrote", out)


if __name__ == "__main__":
    main()
