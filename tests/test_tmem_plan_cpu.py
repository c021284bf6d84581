"""Host arithmetic that keeps tensor memory from deadlocking the scoring kernels (csrc/tmem_plan.h):
over every shape the launchers can produce, the CTAs that fit on a multiprocessor by shared memory must
never ask for more than its 512 tensor-memory columns together.  Checked by a small C++ program built
from the header itself (no GPU needed)."""
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PROGRAM = r"""
#include <cstdio>
#include "tmem_plan.h"
using namespace mvla;
int main()
{
    int checked = 0, padded = 0;
    for (int esize = 1; esize <= 2; ++esize)
        for (int head_dim = 64; head_dim <= 256; head_dim += 32)
            for (int tiles = 1; tiles <= 4; ++tiles)                 // 4096 visual tokens / 128 / cluster of 8
                for (int npad = 16; npad <= 64; npad += 16) {
                    const int tcol = npad <= 16 ? 16 : (npad <= 32 ? 32 : 64);
                    const int cols = tmem_cols_for(tiles * tcol);
                    const size_t khalves = (head_dim * esize + 127) / 128;
                    const size_t dyn = 1024 + khalves * (static_cast<size_t>(tiles) * 16384 + npad * 128);
                    if (dyn > 227 * 1024) continue;                  // refused by the launcher before this point
                    const size_t got = smem_for_tmem(dyn, cols);
                    if (got == 0 || got < dyn || got > static_cast<size_t>(kSmemMaxPerCta)) { std::printf("bad size %zu\n", got); return 1; }
                    if (ctas_by_smem(got) * cols > kTmemColsPerSm) { std::printf("over-subscribed\n"); return 1; }
                    // the padding is the smallest that works: one CTA fewer would still have fitted the columns
                    if (got > dyn && (ctas_by_smem(got) + 1) * cols <= kTmemColsPerSm) { std::printf("padded too far\n"); return 1; }
                    padded += got > dyn;
                    ++checked;
                }
    // the shape the advisory named: 128-byte key rows, 3 tiles, more than 32 queries -> 256 columns, 65 KB
    if (ctas_by_smem(smem_for_tmem(1024 + 1 * (3 * 16384 + 64 * 128), tmem_cols_for(3 * 64))) * 256 > 512) return 1;
    if (tmem_cols_for(1) != 32 || tmem_cols_for(33) != 64 || tmem_cols_for(512) != 512) return 1;
    if (smem_for_tmem(40000, 1024) != 0) return 1;
    std::printf("%d %d\n", checked, padded);
    return 0;
}
"""


def test_resident_ctas_never_oversubscribe_tensor_memory(tmp_path):
    src = tmp_path / "plan.cpp"
    src.write_text(PROGRAM)
    exe = tmp_path / "plan"
    subprocess.run(["g++", "-std=c++17", "-O1", "-I", os.path.join(ROOT, "paper_2604_09244_b200", "csrc"),
                    "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    checked, padded = int(out[0]), int(out[1])
    assert checked > 150 and padded > 0          # the grid was walked, and the guard had something to do
