"""Reader of the hand-worked tree-sizing cases under tests/golden/ (cast_step_*.txt).

Only parsing: the expected values are the ones written (with their derivation)
in the text files; nothing here computes any quantity of the method.
"""
from __future__ import annotations

import os
from fractions import Fraction

import numpy as np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ZERO_PROB_LOGIT = -1000.0  # exp() of it is exactly 0 in fp64 and fp32


def _frac(tok: str) -> Fraction:
    return Fraction(tok)


def _rows(text: str):
    """'1 2 ; 3 4' -> [[1, 2], [3, 4]] as Fractions."""
    return [[_frac(t) for t in part.split()] for part in text.split(";")]


class GoldenCase:
    def __init__(self, name):
        self.name = name
        self.param = {}
        self.root = None
        self.kv_len = None
        self.fT = {}
        self.fD = {}
        self.rows = {}  # (layer, b, r) -> [p0..pV-1] numerators over 16
        self.expect = {}  # tuple of key words -> list of rows of Fractions

    # ---- inputs -----------------------------------------------------------
    @property
    def B(self):
        return len(self.root)

    def logits(self, layer: int) -> np.ndarray:
        """[B, W, V] float64 logits = log(probability); rows not listed are zeros."""
        V, W = int(self.param["V"]), int(self.param["W"])
        x = np.zeros((self.B, W, V), dtype=np.float64)
        for (l, b, r), p in self.rows.items():
            if l == layer:
                x[b, r] = [np.log(float(v) / 16.0) if v > 0 else ZERO_PROB_LOGIT for v in p]
        return x

    def table_arrays(self):
        M, Ntab = int(self.param["M"]), int(self.param["Ntab"])
        fT = np.array([[float(v) for v in self.fT[g]] for g in range(1, M + 1)], dtype=np.float64)
        fD = np.array([[float(v) for v in self.fD[g]] for g in range(1, M + 1)], dtype=np.float64)
        assert fT.shape == (M, Ntab) and fD.shape == (M, Ntab)
        return int(self.param["L"]), M, Ntab, fT, fD

    def config_kwargs(self, **over):
        p = self.param
        kw = dict(vocab=int(p["V"]), top_k=int(p["K"]), max_width=int(p["W"]), max_depth=int(p["H"]),
                  total_token=int(p.get("m", 1)), max_tree=int(p["Ncap"]), fifo_len=int(p.get("R", 8)),
                  C1=float(p.get("C1", 1)), C2=float(p.get("C2", 1)), C3=float(p.get("C3", 1)),
                  enable_bp=int(p.get("bp", 1)), enable_dp=int(p.get("dp", 1)), enable_dr=int(p.get("dr", 1)))
        kw.update(over)
        return kw

    # ---- expectations -----------------------------------------------------
    def get(self, *key):
        return self.expect[tuple(str(k) for k in key)]

    def has(self, *key):
        return tuple(str(k) for k in key) in self.expect

    def ints(self, *key):
        return [[int(v) for v in row] for row in self.get(*key)]

    def steps(self):
        return sorted({int(k[1]) for k in self.expect if k[0] == "step"})

    def layers(self, step):
        return sorted({int(k[3]) for k in self.expect if k[0] == "step" and k[1] == str(step) and k[2] == "layer"})

    def select_budgets(self):
        return sorted({int(k[2]) for k in self.expect if k[0] == "select"})


def load(fname: str):
    """Returns the cases of one golden file in order (a file without 'case' lines is one case)."""
    cases = [GoldenCase(os.path.splitext(fname)[0])]
    started = False
    with open(os.path.join(GOLDEN, fname)) as f:
        for ln in f:
            ln = ln.split("#", 1)[0].strip()
            if not ln:
                continue
            if ln.startswith("case "):
                if started:
                    cases.append(GoldenCase(ln[5:].strip()))
                else:
                    cases[0].name = ln[5:].strip()
                started = True
                continue
            started = True
            c = cases[-1]
            if ln.startswith("param "):
                _, k, v = ln.split()
                c.param[k] = _frac(v)
                continue
            head, vals = [s.strip() for s in ln.split("|")]
            words = head.split()
            if words[0] == "root":
                c.root = [int(v) for v in vals.split()]
            elif words[0] == "kv_len":
                c.kv_len = [int(v) for v in vals.split()]
            elif words[0] in ("fT", "fD"):
                getattr(c, words[0])[int(words[1])] = [_frac(v) for v in vals.split()]
            elif words[0] == "row":
                c.rows[(int(words[1]), int(words[2]), int(words[3]))] = [_frac(v) for v in vals.split()]
            else:
                c.expect[tuple(words)] = _rows(vals)
    return cases
