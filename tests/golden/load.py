"""Reader for the small "key value" text fixtures in this folder."""
import os


def load(name: str) -> dict:
    out = {}
    with open(os.path.join(os.path.dirname(__file__), name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v)
    return out
