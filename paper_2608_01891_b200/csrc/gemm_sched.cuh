// The few-tiles schedule shared by the tcgen05 GEMM kernels: how a list of output tiles, each a run of K steps,
// is dealt to the persistent CTAs so that every CTA streams the same number of weight bytes.
//
// tiles = W * G + R for G CTAs.  The R remainder tiles (ids 0 .. R-1) are cut along K into one equal, contiguous
// share of K steps per CTA and come FIRST; then every CTA takes its W whole tiles (ids R + cta + i * G).  A
// remainder tile whose K range is spread over several CTAs is finished by those CTAs together (each parks an
// fp32 partial; the pieces are summed in CTA order).
#pragma once

namespace aflex {

// One unit of work for a CTA: K blocks [kb0, kb1) of one tile.  slot >= 0 => the unit does not
// cover the whole K range and its partial accumulator goes to partial slot `slot` of this CTA.
struct WorkUnit {
    int tile, kb0, kb1, slot;
};

// Shape of the schedule, identical for every CTA and role.
struct Schedule {
    int kblocks;
    int G;        // CTAs that take whole tiles
    int R;        // remainder tiles (ids 0..R-1), shared along K
    int Gr;       // CTAs that take a share of the remainder (every share non-empty)
    int W;        // whole tiles per CTA (ids R + cta + i*G)
    long long Ur; // R * kblocks
    __device__ Schedule(int kblocks_, int streamk, int total_tiles, int grid) {
        kblocks = kblocks_;
        G = grid;
        if (!streamk) { R = 0; W = (total_tiles + grid - 1) / grid; }
        else { W = total_tiles / grid; R = total_tiles - W * grid; }
        Ur = (long long)R * kblocks;
        Gr = (int)(Ur < G ? Ur : G);
        total = total_tiles;
    }
    int total;
    __device__ long long share_begin(int c) const { return Ur * c / Gr; }
    // CTA whose remainder share contains unit position x
    __device__ int cta_of(long long x) const {
        int c = (int)((x * Gr) / Ur);
        if (c >= Gr) c = Gr - 1;
        while (c > 0 && share_begin(c) > x) --c;
        while (c + 1 < Gr && share_begin(c + 1) <= x) ++c;
        return c;
    }
};

// Walks the units of CTA `cta` in order; every role of the CTA walks the same sequence.
struct UnitCursor {
    const Schedule& sc;
    int cta;
    long long u, u_end;   // position in the remainder unit list
    int i;                // index of the next whole tile
    bool first;
    __device__ UnitCursor(const Schedule& s, int cta_) : sc(s), cta(cta_), i(0), first(true) {
        if (cta < sc.Gr) { u = sc.share_begin(cta); u_end = sc.share_begin(cta + 1); }
        else { u = 0; u_end = 0; }
    }
    __device__ bool next(WorkUnit& out) {
        if (u < u_end) {
            out.tile = (int)(u / sc.kblocks);
            out.kb0 = (int)(u % sc.kblocks);
            out.kb1 = (int)min((long long)sc.kblocks, out.kb0 + (u_end - u));
            const bool whole = out.kb0 == 0 && out.kb1 == sc.kblocks;
            // at most two partial units per CTA: the first unit of its share (slot 0) and a later one (slot 1)
            out.slot = whole ? -1 : (first ? 0 : 1);
            first = false;
            u += out.kb1 - out.kb0;
            return true;
        }
        const int t = sc.R + cta + i * sc.G;
        if (i >= sc.W || t >= sc.total) return false;
        ++i;
        out.tile = t; out.kb0 = 0; out.kb1 = sc.kblocks; out.slot = -1;
        return true;
    }
};

}  // namespace aflex
