"""Writes tests/golden/index_examples.txt: index -> class and coordinates, as the CPU oracle decodes
them under the index order this build reads into the paper's Sec. 2.1 (the paper prints no example of
its own).  Calls nothing but oracle/.  Run: python tests/golden/make_index_examples.py"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import oracle as O  # noqa: E402

N = O.total_points()
INDICES = [0, 1, 1103, 1104, 1105, 98_256, 196_559, 196_560, 16_969_680, 415_003_680, 12_345_678_901_234,
           40_556_880_458_640, N // 3, N // 2, N - 4097, N - 1]

with open(os.path.join(HERE, "index_examples.txt"), "w") as f:
    f.write("# index <tab> class <tab> 24 coordinates; written by make_index_examples.py from oracle/ alone\n")
    for i in INDICES:
        c, x = O.decode(i)
        f.write(f"{i}\t{c}\t{' '.join(str(int(v)) for v in x)}\n")
print("wrote", len(INDICES), "examples")
