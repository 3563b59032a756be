"""Reader for tests/golden/early_pruning_order.txt (a hand-worked GreedyEarlyPruning instance)."""
import os
import re

import numpy as np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_early_pruning_instance():
    """Returns (instance dict, list of cases); a case = {policy, accounting, E: {k: set of 1-based
    tuples}, visible: {(k, layer, head): [source scales]}}."""
    inst = {"scas": {}, "cas": {}}
    cases = []
    cur = None
    for raw in open(os.path.join(GOLDEN, "early_pruning_order.txt")):
        line = raw.split("#")[0].strip()
        if not line:
            continue
        w = line.split()
        if w[0] == "sides":
            inst["sides"] = [int(x) for x in w[1:]]
        elif w[0] in ("L", "H", "s", "B"):
            inst[w[0]] = int(w[1])
        elif w[0] == "b":
            inst["b"] = float(w[1])
        elif w[0] == "N":
            inst["N"] = [int(x) for x in w[1:]]
        elif w[0] == "scas":
            inst["scas"][int(w[1])] = [float(x) for x in w[2:]]
        elif w[0] == "cas":
            inst["cas"][int(w[1])] = float(w[2])
        elif w[0] == "policy":
            cur = {"policy": w[1], "accounting": w[2], "E": {}, "visible": {}}
            cases.append(cur)
        elif w[0] == "E":
            k = int(w[1])
            cur["E"][k] = {tuple(int(x) for x in m) for m in re.findall(r"\((\d+)(?:,(\d+))?(?:,(\d+))?\)", line)
                           for m in [[y for y in m if y != ""]]}
        elif w[0] == "visible":
            k = int(w[1])
            layer, head = (int(x) for x in re.search(r"\((\d+),(\d+)\)", line).groups())
            cur["visible"][(k, layer, head)] = [int(x) for x in line.split(":")[1].split()]
        else:
            raise ValueError(line)
    L, H, K = inst["L"], inst["H"], len(inst["sides"])
    scas = np.zeros((L, H, K))
    cas = np.zeros((L, H))
    for flat, vals in inst["scas"].items():
        scas[flat // H, flat % H, inst["s"]:inst["s"] + len(vals)] = vals
    for flat, v in inst["cas"].items():
        cas[flat // H, flat % H] = v
    inst["scas_array"], inst["cas_array"] = scas, cas
    return inst, cases
