"""Host logic of the look-up-table launch: the cut of the task space into one share per CTA (csrc/bpdq_partition.h).
The header is plain C++; a small driver is compiled with g++ and its cuts are checked against what a cut must satisfy
and against a brute-force optimum on tiny cases."""
import itertools
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER_DIR = os.path.join(ROOT, "paper_2602_04163_b200", "csrc")

DRIVER = r"""
#include <cstdio>
#include <cstdlib>
#include "bpdq_partition.h"
// argv: grid cost n nrg_0 nslices_0 ... ; prints dearest share cost, then t_begin[0..grid]
int main(int argc, char** argv) {
    const int grid = atoi(argv[1]), cost = atoi(argv[2]), n = atoi(argv[3]);
    int nrg[16], nsl[16];
    for (int k = 0; k < n; ++k) { nrg[k] = atoi(argv[4 + 2 * k]); nsl[k] = atoi(argv[5 + 2 * k]); }
    int* t = (int*)malloc(sizeof(int) * (grid + 1));
    const double dearest = bpdq::cut_task_space(nrg, nsl, n, grid, cost, t);
    printf("%.3f", dearest);
    for (int b = 0; b <= grid; ++b) printf(" %d", t[b]);
    printf("\n");
    return 0;
}
"""


@pytest.fixture(scope="module")
def driver(tmp_path_factory):
    d = tmp_path_factory.mktemp("partition")
    src, exe = d / "driver.cpp", d / "driver"
    src.write_text(DRIVER)
    subprocess.run(["g++", "-O2", "-std=c++17", "-I", HEADER_DIR, str(src), "-o", str(exe)], check=True)
    return str(exe)


def cut(driver, grid, cost, linears):
    args = [driver, str(grid), str(cost), str(len(linears))]
    for nrg, nsl in linears:
        args += [str(nrg), str(nsl)]
    out = subprocess.run(args, check=True, capture_output=True, text=True).stdout.split()
    return float(out[0]), [int(v) for v in out[1:]]


def share_costs(t_begin, cost, linears):
    """Cost of every share: its tasks plus `cost` per slice it touches."""
    bounds, t = [], 0                                   # slice boundaries in the concatenated task space
    for nrg, nsl in linears:
        for _ in range(nsl):
            bounds.append((t, t + nrg))
            t += nrg
    costs = []
    for a, b in zip(t_begin[:-1], t_begin[1:]):
        touched = sum(1 for lo, hi in bounds if max(a, lo) < min(b, hi))
        costs.append((b - a) + cost * touched)
    return costs, t


def layer(shapes):
    """(row groups, slices) of linears given as (out, in): 16 rows per task, 512 columns per slice."""
    return [(o // 16, (i // 128 + 3) // 4) for o, i in shapes]


LAYER_72B = layer([(8192, 8192), (1024, 8192), (1024, 8192), (8192, 8192), (29568, 8192), (29568, 8192), (8192, 29568)])
LAYER_7B = layer([(3584, 3584), (512, 3584), (512, 3584), (3584, 3584), (18944, 3584), (18944, 3584), (3584, 18944)])


@pytest.mark.parametrize("linears,grid,cost", [
    (LAYER_72B, 148, 48), (LAYER_72B, 148, 96), (LAYER_7B, 148, 48), (layer([(29568, 8192)]), 148, 64),
    (layer([(4096, 4096)]), 148, 64), (layer([(160, 640)]), 20, 64), (layer([(16, 128)]), 1, 64),
    (layer([(8192, 29568), (1024, 8192)]), 132, 32),
])
def test_cut_is_a_partition_and_balanced(driver, linears, grid, cost):
    dearest, t = cut(driver, grid, cost, linears)
    costs, total = share_costs(t, cost, linears)
    assert len(t) == grid + 1 and t[0] == 0 and t[-1] == total
    assert all(a <= b for a, b in zip(t[:-1], t[1:]))                   # contiguous, in order, nothing twice
    assert max(costs) == pytest.approx(dearest, abs=1.0)                # the returned bound is the dearest share's cost
    # no cut can do better than an even split of the work plus one set-up per slice and per cut
    nslices = sum(nsl for _, nsl in linears)
    lower = (total + cost * nslices) / grid
    if total >= 8 * grid:                                               # enough work for every CTA
        assert max(costs) <= 1.08 * lower + 2 * cost


def test_cut_matches_brute_force_on_tiny_cases(driver):
    """All contiguous cuts of a tiny task space: the header's cut must reach the best possible dearest share
    (up to the rule that a share is not opened into a slice for fewer than eight tasks, which tiny slices never meet)."""
    for linears, grid, cost in [([(5, 2), (3, 1)], 3, 4), ([(7, 1), (2, 3)], 4, 2), ([(4, 4)], 5, 3)]:
        dearest, t = cut(driver, grid, cost, linears)
        costs, total = share_costs(t, cost, linears)
        best = min(max(share_costs([0, *c, total], cost, linears)[0])
                   for c in itertools.combinations_with_replacement(range(total + 1), grid - 1))
        assert max(costs) <= best + 1, (linears, grid, cost, t, best)
