"""Writes tests/golden/lloyd_max_d<dim>_b6.txt: the 64 centroids of the 6-bit Lloyd-Max codebook of Eq. 3 for the
sphere marginal of Eq. 2, as computed by the oracle alone (minutes per width, hence stored).

    python tests/golden/make_codebook_b6.py 3072 5120

One value per line, repr of a float64, ascending.  Boundaries are the midpoints of neighbours (Eq. 3).
"""
import os
import sys

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", ".."))
from oracle import codebook as ocb  # noqa: E402

if __name__ == "__main__":
    for arg in sys.argv[1:]:
        dim = int(arg)
        cb = ocb.lloyd_max(dim, 6)
        path = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"lloyd_max_d{dim}_b6.txt")
        with open(path, "w") as f:
            f.write(f"# 6-bit Lloyd-Max centroids for f_d, d = {dim} (Eq. 2-3); written by make_codebook_b6.py from oracle.codebook\n")
            for c in cb.centroids:
                f.write(repr(float(c)) + "\n")
        print("wrote", path)
