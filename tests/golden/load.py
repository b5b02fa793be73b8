"""Reader for the small text fixtures in this folder."""
import os


def paper_constants():
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "paper_constants.txt")) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            name, value = line.split()
            out[name] = float(value)
    return out
