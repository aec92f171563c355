"""Host logic of the prefill GEMM's scheduler: `csrc/aq_gemm_runs.h` (how the (row tile, token super-tile, k-slab)
work is cut into one contiguous run per CTA), compiled with the host compiler alone and driven from a small C++
program.  Checked for many shapes: the bounds partition the work (ascending, even, first 0, last total), the run that
holds a tile's last slab starts inside that tile or covers the tile whole (what the store-first protocol of the kernel
relies on), and the most expensive run is never more expensive than under the equal cut it replaced."""
import os
import shutil
import subprocess
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HDR = os.path.join(ROOT, "paper_2605_24011_b200", "csrc")

SRC = textwrap.dedent(r"""
    #include <algorithm>
    #include <cstdio>
    #include <vector>
    #include "aq_gemm_runs.h"
    using namespace aq;
    #define CHECK(c) do { if (!(c)) { std::printf("FAIL line %d: %s (n_slabs %lld R %lld M %d grid %d)\n", __LINE__, #c, n_slabs, R, M, grid); return 1; } } while (0)

    // the same derivation of the tile structure as the launcher's
    static int one(long long n_slabs, long long R, int M, int grid) {
        long long n_st, n2;
        if (M > 256) { n_st = (M + 511) / 512; n2 = (M - 512 * (n_st - 1) > 256) ? n_st : n_st - 1; }
        else { n_st = 1; n2 = 0; }
        const long long c2 = 2 * n_slabs, c1 = n_slabs, n_two = n2 * R;
        const long long total = n_slabs * R * (2 * n2 + (n_st - n2));
        if (total / 2 < grid) grid = (int)(total / 2);
        if (grid < 1) return 0;
        std::vector<int> b(grid + 1, -1);
        cut_runs(total, n_two, c2, c1, grid, b.data());
        CHECK(b[0] == 0 && b[grid] == total);
        long long worst = 0;
        for (int c = 0; c < grid; ++c) {
            CHECK(b[c] <= b[c + 1] && b[c] % 2 == 0);
            worst = std::max(worst, run_cost(b[c], b[c + 1], n_two, c2, c1));
        }
        // a run that contains a tile's last unit and does not start inside that tile covers the tile whole
        const long long reg2 = n_two * c2;
        for (int c = 0; c < grid; ++c) {
            for (long long pos = b[c]; pos < b[c + 1];) {
                const long long ts = pos < reg2 ? pos / c2 * c2 : reg2 + (pos - reg2) / c1 * c1;
                const long long te = ts + (pos < reg2 ? c2 : c1);
                if (te <= b[c + 1] && ts < b[c]) CHECK(pos == b[c]);          // the tile's tail: first thing of the run
                pos = std::min<long long>(te, b[c + 1]);
            }
        }
        // never worse than equal runs
        long long worst_equal = 0;
        for (int c = 0; c < grid; ++c) {
            const long long lo = (total * c / grid) & ~1LL, hi = (c + 1 == grid) ? total : ((total * (c + 1) / grid) & ~1LL);
            worst_equal = std::max(worst_equal, run_cost(lo, hi, n_two, c2, c1));
        }
        CHECK(worst <= worst_equal);
        // and no run costs more than the work spread evenly plus what one tile and its pieces can add
        CHECK(worst <= total / grid + c2 + 4 * GM_SEG_COST + 2 || worst <= worst_equal);
        return 0;
    }

    int main() {
        const int Ms[] = {9, 16, 50, 130, 200, 256, 257, 300, 512, 513, 768, 1000, 1024, 4096};
        const long long Ks[] = {256, 1024, 4096, 11008, 16384};
        const long long Ns[] = {16, 128, 1000, 1024, 2048, 4096, 11008, 12288, 22016, 65536};
        const int grids[] = {1, 7, 132, 148, 160, 192};
        int n = 0;
        for (int M : Ms) for (long long K : Ks) for (long long N : Ns) for (int g : grids) {
            const long long n_slabs = (K + 255) / 256 * 2, R = (N + 127) / 128;
            if (n_slabs * R * 16 > 2000000000LL) continue;
            if (one(n_slabs, R, M, g)) return 1;
            ++n;
        }
        std::printf("OK %d\n", n);
        return 0;
    }
""")


@pytest.mark.skipif(shutil.which("g++") is None, reason="no host compiler")
def test_gemm_runs_partition(tmp_path):
    src = tmp_path / "runs.cpp"
    exe = tmp_path / "runs"
    src.write_text(SRC)
    subprocess.run(["g++", "-std=c++17", "-O1", "-I", HDR, str(src), "-o", str(exe)], check=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.startswith("OK")
