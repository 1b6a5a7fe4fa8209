"""Reader for the plain-text fixtures under tests/golden/."""
import os


def read_golden(name):
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
    out = {}
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(":")
            out[key.strip()] = [float(x) if ("." in x or "e" in x) else int(x) for x in rest.split()]
    return out
