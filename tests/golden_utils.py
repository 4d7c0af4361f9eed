"""Reader of the hand-worked rebalancing plans in tests/golden/plan_handworked.txt."""
import os

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_plan_cases():
    """One dict per case: the file's fields as strings, plus parsed ``counts_i``, ``mask_i``,
    ``moves_t`` [(expert, src, dst, rows)], ``before_i`` and ``after_i``."""
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "plan_handworked.txt")):
        line = line.split("#")[0].rstrip("\n")
        if "=" not in line:
            continue
        k, v = [s.strip() for s in line.split("=", 1)]
        if k == "case":
            cur = {"case": v}
            cases.append(cur)
        else:
            cur[k] = v
    for c in cases:
        c["counts_i"] = [int(v) for v in c["counts"].split()]
        c["mask_i"] = [int(v) for v in c["mask"].split()]
        moves = []
        for m in c["moves"].split():
            e, sd, rows = m.split(":")
            s, dd = sd.split(">")
            moves.append((int(e), int(s), int(dd), int(rows)))
        c["moves_t"] = moves
        c["before_i"] = [int(v) for v in c["load_before"].split()]
        c["after_i"] = [int(v) for v in c["load_after"].split()]
    return cases
