"""Glue used by the tests only: moves metadata from the oracle's struct to the library's handle
(plain table copies, no arithmetic)."""
import numpy as np


def lib_meta_from_oracle(binding, ometa):
    """The oracle's metadata handed to the library (the library re-derives its own codes and tables)."""
    return binding.ecco_meta_create(ometa.S, ometa.e, ometa.patterns(), ometa.cb_lengths(), ometa.kp_lengths())


def oracle_meta_from_lib(eo, lmeta):
    S, e, pat, cb, kp = lmeta.tables()
    m = eo.Meta()
    m.S, m.H, m.e = S, 4, e
    pu = pat.view(np.uint16)
    for k in range(S):
        m.kp_len[k] = int(kp[k])
        for j in range(15):
            m.pattern[k][j] = int(pu[k, j])
        for h in range(4):
            for s in range(16):
                m.cb_len[k][h][s] = int(cb[k, h, s])
    return m


# Largest errors the fused calls showed in this run, per label: {label: [max |y - ref| / sum|w x|, max plain relative
# error where |ref| >= 0.1 rms]}.  conftest.py prints them at the end of the session.
FUSED_MAXIMA = {}


def record_fused(label, scaled, plain):
    a, b = FUSED_MAXIMA.get(label, (0.0, 0.0))
    FUSED_MAXIMA[label] = (max(a, float(scaled)), max(b, float(plain)))
