"""Reader for the small text fixtures under tests/golden/."""
import os
from fractions import Fraction as Fr

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_printed(name):
    """Parse '[name rows cols]' sections of rationals and the '[errata]' list."""
    mats, errata, cur, want = {}, [], None, None
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("["):
                head = line.strip("[]").split()
                cur = head[0]
                if cur == "errata":
                    want = None
                else:
                    want = (int(head[1]), int(head[2]))
                    mats[cur] = []
                continue
            if cur == "errata":
                mname, r, c, printed, fixed = line.split()
                errata.append((mname, int(r), int(c), Fr(printed), Fr(fixed)))
            else:
                row = [Fr(tok) for tok in line.split()]
                assert len(row) == want[1], (name, cur, line)
                mats[cur].append(row)
    for k, v in mats.items():
        assert len(v) > 0, k
    return mats, errata


def read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(tok) for tok in line.split()])
    return rows
