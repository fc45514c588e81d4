"""Writes sweep_shapes.csv: the 2,000-shape dynamic sweep, from the seeded recipe in ``synth``.

Run once: ``python -m paper_2608_10803_b200.data.make_sweep``.  The CSV is committed
so that the list never depends on a platform's floating-point library.
"""
import csv
import os

from paper_2608_10803_b200 import synth


def main():
    shapes, draws = synth.draw_sweep_shapes()
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "sweep_shapes.csv")
    with open(path, "w", newline="") as f:
        w = csv.writer(f)
        w.writerow(["index", "M", "N", "K"])
        for i, (m, n, k) in enumerate(shapes):
            w.writerow([i, m, n, k])
    print(f"{len(shapes)} shapes from {draws} draws -> {path}")
    print("first five:", shapes[:5])


if __name__ == "__main__":
    main()
