// Host-side check of the index arithmetic the kernels share (s2a_params.h): exhaustive on small
// shapes, no GPU.  Prints "ok" and returns 0, or says what failed.
#include <cstdio>
#include <set>
#include <vector>

#include "s2a_params.h"

using namespace s2a;

static int fail(const char* what, int a = 0, int b = 0, int c = 0) {
    std::printf("FAIL %s (%d %d %d)\n", what, a, b, c);
    return 1;
}

static Geometry geometry(int B, int N, int H, int Hkv, int G, int n_unshifted, int shift, int leak_free, int swapped) {
    Geometry g{};
    g.B = B, g.N = N, g.H = H, g.Hkv = Hkv, g.G = G, g.n_unshifted = n_unshifted, g.shift = shift;
    g.groups = N / G, g.leak_free = leak_free, g.swap_wrapped = swapped;
    g.tiles_per_group = 0;
    for (int s : {0, shift})
        for (int grp = 0; grp < g.groups; ++grp) {
            const int n = group_layout(g, s, grp).nTiles;
            if (n > g.tiles_per_group) g.tiles_per_group = n;
        }
    return g;
}

int main() {
    // 1. block order: every (unit, rank) exactly once; inside a chunk of units ranks never decrease
    for (int units : {1, 7, 8, 9, 16, 29})
        for (int tiles : {1, 2, 5, 16}) {
            std::set<std::pair<int, int>> seen;
            int prev_rank = 0, prev_chunk = -1;
            for (long long idx = 0; idx < 1LL * units * tiles; ++idx) {
                int u, r;
                decode_block(idx, units, tiles, &u, &r);
                if (u < 0 || u >= units || r < 0 || r >= tiles) return fail("decode_block range", units, tiles, (int)idx);
                if (!seen.insert({u, r}).second) return fail("decode_block repeats", units, tiles, (int)idx);
                const int chunk = u / kUnitChunk;
                if (chunk == prev_chunk && r < prev_rank) return fail("decode_block rank order", units, tiles, (int)idx);
                if (chunk < prev_chunk) return fail("decode_block chunk order", units, tiles, (int)idx);
                prev_chunk = chunk, prev_rank = r;
            }
        }
    // 2. spill blocks: (unit, j, n) with 2 j <= n < 2 T maps one-to-one onto [0, units * T (T + 1))
    for (int T : {1, 2, 3, 8, 17}) {
        const int units = 3;
        std::vector<char> hit(units * spill_blocks_per_unit(T), 0);
        for (int u = 0; u < units; ++u)
            for (int j = 0; j < T; ++j)
                for (int n = 2 * j; n < 2 * T; ++n) {
                    const long long b = spill_block(u, T, j, n);
                    if (b < 0 || b >= (long long)hit.size() || hit[b]) return fail("spill_block", T, j, n);
                    hit[b] = 1;
                }
        for (char h : hit)
            if (!h) return fail("spill_block leaves a gap", T);
        // the two halves of a query tile are neighbours (the dQ kernel fetches them with one copy)
        for (int j = 0; j < T; ++j)
            for (int i = j; i < T; ++i)
                if (spill_block(1, T, j, 2 * i + 1) != spill_block(1, T, j, 2 * i) + 1) return fail("spill halves", T, j, i);
    }
    // 3. tiles of a group: every rolled position of the group exactly once, in causal order, each tile a
    //    contiguous run of original tokens; variant 3 puts the front tokens first
    struct Shape { int N, G, shift, swapped; };
    for (Shape sh : {Shape{1024, 256, 128, 0}, Shape{2400, 600, 300, 0}, Shape{2400, 600, 300, 1}, Shape{1000, 200, 100, 0},
                     Shape{4096, 1024, 384, 0}, Shape{512, 512, 256, 0}, Shape{1536, 384, -192, 0}}) {
        const Geometry geo = geometry(1, sh.N, 2, 2, sh.G, 1, sh.shift, 0, sh.swapped);
        for (int s : {0, sh.shift})
            for (int grp = 0; grp < geo.groups; ++grp) {
                const GroupLayout L = group_layout(geo, s, grp);
                std::vector<int> order;   // original tokens in the order the tiles present them
                for (int i = 0; i < L.nTiles; ++i) {
                    const TileRef t = tile_ref(L, i);
                    if (t.valid <= 0 || t.valid > kTile) return fail("tile valid", sh.N, grp, i);
                    if (t.tok0 < 0 || t.tok0 + t.valid > sh.N) return fail("tile leaves the sequence", sh.N, grp, i);
                    for (int r = 0; r < t.valid; ++r) order.push_back(t.tok0 + r);
                    int sub = 0;
                    for (int h = 0; h < 2; ++h) {
                        const TileRef st = subtile_ref(L, 2 * i + h);
                        if (st.valid < 0 || st.valid > kSubTile) return fail("subtile valid", sh.N, grp, i);
                        if (st.valid > 0 && st.tok0 != t.tok0 + h * kSubTile) return fail("subtile start", sh.N, grp, i);
                        sub += st.valid;
                    }
                    if (sub != t.valid) return fail("subtiles do not add up", sh.N, grp, i);
                }
                if ((int)order.size() != sh.G) return fail("group size", sh.N, grp, (int)order.size());
                // expected: rolled positions grp G .. (grp + 1) G - 1 are original tokens (x + s) mod N
                std::vector<int> want;
                for (int x = grp * sh.G; x < (grp + 1) * sh.G; ++x) want.push_back(((x + s) % sh.N + sh.N) % sh.N);
                if (L.swapped) {   // front tokens (the part after the wrap) first
                    std::vector<int> w2(want.begin() + L.lenA, want.end());
                    w2.insert(w2.end(), want.begin(), want.begin() + L.lenA);
                    want = w2;
                }
                if (order != want) return fail("token order", sh.N, s, grp);
            }
    }
    std::printf("ok\n");
    return 0;
}
