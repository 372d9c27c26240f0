"""Parser for the small text fixtures under tests/golden/."""
import os
from fractions import Fraction

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _fr(tok):
    return Fraction(tok)


def load_worked_2x4():
    out = dict(sweeps={}, canon={})
    with open(os.path.join(GOLDEN, "worked_2x4.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, _, rest = line.partition(" ")
            if head == "W":
                out["W"] = [[_fr(t) for t in row.split()] for row in rest.split(";")]
            elif head == "X":
                out["x"] = [_fr(t) for t in rest.split()]
            elif head == "Y":
                out["y"] = [_fr(t) for t in rest.split()]
            elif head == "SWEEPS":
                out["n_sweeps"] = int(rest)
            elif head == "WHAT":
                out["What"] = [[_fr(t) for t in row.split()] for row in rest.split(";")]
            elif head == "ETOTAL":
                out["Etotal"] = _fr(rest)
            elif head == "EGLOBAL_ROW1":
                out["Eglobal_row1"] = _fr(rest)
            elif head == "CANON":
                parts = [p.split() for p in rest.split("|")]
                row = int(parts[0][0])
                out["canon"][row] = dict(alpha=(_fr(parts[0][1]), _fr(parts[0][2])),
                                         T1=[int(t) for t in parts[1]], T2=[int(t) for t in parts[2]])
            else:
                parts = [p.split() for p in line.split("|")]
                t, row = int(parts[0][0]), int(parts[0][1])
                out["sweeps"][(t, row)] = dict(alpha=(_fr(parts[0][2]), _fr(parts[0][3])),
                                               T1=[int(v) for v in parts[1]],
                                               T2=[int(v) for v in parts[2]], E=_fr(parts[3][0]))
    return out
