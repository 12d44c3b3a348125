// Retrieval knapsack (paper, Sec. 3.4, Eq. 1-2): which groups to load under a KV-memory budget.
// Host-only: a 0/1 dynamic programme over the quantised budget with a take/skip table for the back-trace.
#include <cstdint>
#include <new>
#include <vector>

#include "../../include/enl.h"

extern "C" int enl_select_knapsack(int32_t n, const float *prob, float threshold, const int64_t *mem_bytes,
                                   int64_t budget_bytes, int64_t quantum, int32_t *sel_out)
{
    if (n < 0 || budget_bytes < 0 || quantum <= 0) return ENL_E_INVAL;
    if (n > 0 && (!prob || !mem_bytes || !sel_out)) return ENL_E_INVAL;
    for (int i = 0; i < n; ++i)
        if (mem_bytes[i] < 0) return ENL_E_INVAL;
    const int64_t cap = budget_bytes / quantum;                         // budget rounded down
    if (cap > (int64_t{1} << 31) || (cap + 1) * static_cast<int64_t>(n) > (int64_t{1} << 33)) return ENL_E_NOMEM;
    try {
        std::vector<double> best(static_cast<size_t>(cap) + 1, 0.0);    // best value with capacity c, groups 0..i
        std::vector<uint8_t> take(static_cast<size_t>(n) * (cap + 1), 0);
        for (int i = 0; i < n; ++i) {
            const double v = static_cast<double>(prob[i]) - static_cast<double>(threshold);
            if (!(v > 0.0)) continue;                                   // never worth its memory
            const int64_t w = (mem_bytes[i] + quantum - 1) / quantum;   // size rounded up
            if (w > cap) continue;
            uint8_t *row = take.data() + static_cast<size_t>(i) * (cap + 1);
            for (int64_t c = cap; c >= w; --c) {
                const double with = best[c - w] + v;
                if (with > best[c]) { best[c] = with; row[c] = 1; }
            }
        }
        int count = 0;
        int64_t c = cap;
        std::vector<int32_t> rev;
        for (int i = n - 1; i >= 0; --i) {
            if (take[static_cast<size_t>(i) * (cap + 1) + c]) {
                rev.push_back(i);
                c -= (mem_bytes[i] + quantum - 1) / quantum;
            }
        }
        for (auto it = rev.rbegin(); it != rev.rend(); ++it) sel_out[count++] = *it;
        return count;
    } catch (const std::bad_alloc &) {
        return ENL_E_NOMEM;
    }
}
