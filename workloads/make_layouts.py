"""Write the committed tensor-size lists under ``workloads/layouts/``.

Run as ``python -m workloads.make_layouts``.  Sizes are drawn once from the layout hash
stream and stored as data so that every consumer reads the same integers.
"""
import json
import os

from .configs import draw_log_uniform_sizes

HERE = os.path.dirname(os.path.abspath(__file__))


def main():
    out = {
        "cfg2": draw_log_uniform_sizes(2, 62, 11_700_000),
        "cfg3": draw_log_uniform_sizes(3, 161, 25_600_000),
        # three dominant FC-like tensors, then 29 log-uniform ones (tensor numbers 3..31)
        "cfg4": [102_760_448, 16_777_216, 4_096_000]
                + draw_log_uniform_sizes(4, 29, 138_000_000 - 123_633_664, first_tensor=3),
    }
    for name, sizes in out.items():
        path = os.path.join(HERE, "layouts", name + ".json")
        with open(path, "w") as f:
            json.dump({"name": name, "n_tensors": len(sizes), "P": sum(sizes), "sizes": sizes}, f)
            f.write("\n")
        print(name, len(sizes), sum(sizes), min(sizes), max(sizes))


if __name__ == "__main__":
    main()
