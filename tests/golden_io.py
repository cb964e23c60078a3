"""Reader for the plain-text worked-example fixtures under tests/golden/."""
from __future__ import annotations

import os
from typing import Dict, List


def _vec(text: str) -> List[float]:
    return [float(t) for t in text.split()]


def _mat(text: str) -> List[List[float]]:
    return [_vec(r) for r in text.split(";")]


def read_records(path: str) -> List[Dict[str, str]]:
    records, cur = [], {}
    with open(path) as fh:
        for line in fh:
            line = line.rstrip("\n")
            if line.startswith("#"):
                continue
            if not line.strip():
                if cur:
                    records.append(cur)
                    cur = {}
                continue
            key, _, val = line.partition("=")
            cur[key.strip()] = val.strip()
    if cur:
        records.append(cur)
    return records


def worked_examples(golden_dir: str):
    out = []
    for rec in read_records(os.path.join(golden_dir, "worked_examples.txt")):
        case = {"name": rec["name"], "op": rec["op"], "x": _mat(rec["x"]),
                "expect": _mat(rec["expect"]), "derivation": rec["derivation"]}
        for key in ("gamma", "beta", "weight"):
            if key in rec:
                case[key] = _vec(rec[key])
        if "additive" in rec:
            case["additive"] = _mat(rec["additive"])
        case["eps"] = float(rec.get("eps", "0"))
        case["causal_period"] = int(rec.get("causal_period", "0"))
        case["skip_rows"] = [int(t) for t in rec.get("skip_rows", "").split()]
        out.append(case)
    return out
