// Host arithmetic that keeps tensor memory from deadlocking the scoring kernels.
//
// A multiprocessor has 512 columns of tensor memory.  tcgen05.alloc blocks until its columns are free, and
// the scoring kernels hold their columns while they wait for the other CTAs of their cluster.  If the CTAs
// that fit on a multiprocessor by registers, threads and shared memory could together ask for more than
// 512 columns, this cycle is possible: CTA A holds columns on SM X and waits for its peer A' on SM Y; A' is
// blocked in the allocation behind CTA B, which waits for its peer B', blocked in the allocation on SM X
// behind A.  No bounded mbarrier wait can break it.  So the launchers make sure that
//     resident CTAs per multiprocessor x columns per CTA <= 512
// by asking for enough dynamic shared memory that no more CTAs than that fit, and check the result with the
// occupancy calculator before every launch configuration is used.
#pragma once

#include <stddef.h>

namespace mvla {

constexpr int kTmemColsPerSm = 512;
constexpr int kSmemPerSm = 233472;          // 228 KB of shared memory per multiprocessor
constexpr int kSmemReservedPerCta = 1024;   // taken by the system for every resident CTA
constexpr int kSmemMaxPerCta = 232448;      // 227 KB: the most one CTA may ask for

// Columns tcgen05.alloc is asked for: a power of two, at least 32.
inline int tmem_cols_for(int columns_needed)
{
    int c = 32;
    while (c < columns_needed) c <<= 1;
    return c;
}

// CTAs that fit on a multiprocessor by shared memory alone (static shared memory counted as zero: the real
// number can only be smaller).
inline int ctas_by_smem(size_t dyn_smem)
{
    return static_cast<int>(kSmemPerSm / (dyn_smem + kSmemReservedPerCta));
}

// Dynamic shared memory to launch with: `dyn_smem` or, when that would let too many CTAs share the tensor
// memory, the smallest size that rules the surplus CTA out.  0: no size does (cannot happen for <= 512 columns).
inline size_t smem_for_tmem(size_t dyn_smem, int tmem_cols)
{
    if (tmem_cols > kTmemColsPerSm) return 0;
    const int max_ctas = kTmemColsPerSm / tmem_cols;
    if (ctas_by_smem(dyn_smem) <= max_ctas) return dyn_smem;
    const size_t footprint = kSmemPerSm / (max_ctas + 1) + 1;      // (max_ctas + 1) of these do not fit
    const size_t padded = footprint - kSmemReservedPerCta;
    return padded <= static_cast<size_t>(kSmemMaxPerCta) ? padded : 0;
}

}  // namespace mvla
