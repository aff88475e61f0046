// Host-side planner of the grouped tensor-core kernel's phase-2 chunk list (pure C++, no CUDA).
//
// A launch has n_units units = (expert, 128 intermediate rows). Phase 1 of a unit (gate / up rows)
// runs on CTA unit % grid. Phase 2 (the W_down tile: n_dt pipeline stages, one per 128 output
// columns) can be cut anywhere between d-tiles and run on any CTA once the unit's A^T exists; the
// kernel's CTAs take chunks from this list in order, whoever is free. Chunks are listed in unit
// order (so the units whose phase 1 ends first come first) and get finer towards the end of the
// list ("guided" sizes: about 1 / (2 grid) of what is left, never fewer than kGgMinChunk d-tiles
// while a unit has that many left), so that all CTAs run out of work at about the same time
// even when there are fewer or only slightly more units than CTAs.
#pragma once

#include <algorithm>
#include <cstdint>
#include <vector>

namespace spm {

struct GgTaskHost {      // same layout as the device-side GgTask
    int32_t unit;
    int16_t dt0, dt1;    // phase 2 of d-tiles dt0 .. dt1-1
};

constexpr int kGgMinChunk = 4;    // a chunk also fetches the unit's A^T (16 KB): keep that a small share of its bytes

inline void gg_plan_chunks(int n_units, int n_dt, int grid, std::vector<GgTaskHost>& chunks) {
    chunks.clear();
    long long remaining = static_cast<long long>(n_units) * n_dt;
    for (int u = 0; u < n_units; ++u) {
        int dt = 0;
        while (dt < n_dt) {
            const long long guided = (remaining + 2LL * grid - 1) / (2LL * grid);
            int n = static_cast<int>(std::max<long long>(kGgMinChunk, std::min<long long>(guided, n_dt)));
            n = std::min(n, n_dt - dt);
            if (n_dt - dt - n > 0 && n_dt - dt - n < kGgMinChunk) n = n_dt - dt;     // no sliver at the end of a unit
            chunks.push_back(GgTaskHost{u, static_cast<int16_t>(dt), static_cast<int16_t>(dt + n)});
            dt += n;
            remaining -= n;
        }
    }
}

}  // namespace spm
