"""Readers for the small text fixtures under tests/golden/ (shared by the oracle pins and the GPU parity tests)."""
import os

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for ln in f:
            ln = ln.strip()
            if ln and not ln.startswith("#"):
                yield [p.strip() for p in ln.split(";")]


def layer_budget_cases():
    out = []
    for k_p, beta, bnd, prof, exp in _lines("layer_budgets.txt"):
        prof = [float(x) for x in prof.split(",")]
        b = {int(x) for x in bnd.split(",")}
        out.append(dict(k_p=int(k_p), beta=float(beta), importance=prof,
                        is_boundary=[l in b for l in range(len(prof))],
                        expected=[int(x) for x in exp.split(",")]))
    return out


def _rep(field, conv):
    vals, rep = field.split("x")
    return [conv(v) for v in vals.split(",")] * int(rep)


def head_budget_cases():
    out = []
    for k_l, alpha, n, mp, mm, exp in _lines("head_budgets.txt"):
        out.append(dict(k_l=int(k_l), alpha=float(alpha), n=int(n), mass_p=_rep(mp, float),
                        mass_m=_rep(mm, float), expected=_rep(exp, int)))
    return out
