"""Parser for tests/golden/table1_table2_constants.txt (values the paper prints)."""
import os
from fractions import Fraction


def _parse_value(text: str):
    text = text.strip()
    if text.startswith("0x"):
        return int(text, 16)
    if "* 2^" in text:
        mant, exp = text.split("* 2^")
        return Fraction(mant.strip()) * Fraction(2) ** int(exp)
    try:
        return int(text)
    except ValueError:
        return Fraction(text)


def load(golden_dir: str) -> dict:
    out = {}
    with open(os.path.join(golden_dir, "table1_table2_constants.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            body = line.split(";")[0]
            key, val = body.split("=", 1)
            out[key.strip()] = _parse_value(val)
    return out
