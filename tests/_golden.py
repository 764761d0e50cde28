"""Reader for the text fixtures under tests/golden/."""
import os

GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_hand_example():
    """{(beta, step, array name, worker): [4 values]} from hand_example_n2_d4.txt."""
    rows = {}
    with open(os.path.join(GOLDEN_DIR, "hand_example_n2_d4.txt")) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            p = ln.split()
            rows[(float(p[0]), int(p[1]), p[2], int(p[3]))] = [float(v) for v in p[4:]]
    return rows
