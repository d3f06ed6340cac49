// Work lists of the tensor-core grouped GEMMs, built on the device from the per-expert counts.
#pragma once

#include "moe_internal.h"

namespace lexi {

constexpr int kMaxBalanceTiles = 2048;   // most null tiles the balancing of list 2 may add

struct TileBuildArgs {
    const int32_t *counts, *offsets;
    int32_t E, T, has_shared;
    int32_t feat1, N1_routed, N1_shared, K1;                     // phase 1: features per tile, I, I_s, d
    int32_t bn2, N2, K2_routed, K2_shared;                       // phase 2: BN, d, I, I_s
    int32_t ksplit_routed, kchunk_routed, ksplit_shared, kchunk_shared;
    Tile *tiles1, *tiles2;
    int32_t *n_tiles;
    int32_t cap1, cap2;
    int32_t *status;
    // direct = 1 (T <= 128): phase 1 reads all T token rows of x for every touched expert (one
    // row block per group, rows = T); the epilogue places each row through the position table
    int32_t direct;
    int32_t tile_rows;   // rows of one tile: 128, or 256 when a CTA pair shares a tile
    // rr2 > 0: list 2 is consumed round-robin by rr2 CTAs (or CTA pairs) and the shared expert's tiles
    // reduce over a longer K than the routed ones; null tiles (rows = 0) are slipped in behind the
    // shared tiles so that every consumer ends up with the same amount of work
    int32_t rr2;
    // quotients the host knows (an integer division on the device is a chain of ~30 instructions):
    // feature blocks of phase 1 per routed / shared group, output blocks of phase 2, log2(tile_rows),
    // and how many rounds of short tiles one long shared tile of phase 2 is worth, less one
    int32_t n1_routed_blocks, n1_shared_blocks, n2_blocks, tile_shift, long_over_short_m1;
    int32_t *stats;   // stats[0] += routed experts that received at least one token; stats[1], stats[2] += token
                      // rows the MMAs of this call execute for the routed / shared groups (valid rows rounded up to
                      // the MMA heights the kernels use): executed = padded work, against T k_l and T algorithmic rows
};

// Shared-memory scratch of build_tiles_block.
struct TileBuildSmem {
    int32_t pre1[kMaxExperts + 2], pre2[kMaxExperts + 2];
    int32_t part1[32], part2[32];
};

// Called by all threads of one block; cnt_s/off_s hold counts and offsets in shared memory.
// Group order: the shared expert first (its tiles are always full), then experts 0..E-1.
// Inside a group: 128-row block outermost, then output-feature block, then K slab.
// Several blocks may share the work: block `rank` of `n_blocks` writes every n_blocks-th stripe of
// the lists (each block recomputes the small prefix); rank 0 publishes the tile counts.
__device__ __forceinline__ void build_tiles_block(const TileBuildArgs &a, const int32_t *cnt_s,
                                                  const int32_t *off_s, TileBuildSmem &sm,
                                                  int rank = 0, int n_blocks = 1) {
    const int groups = a.E + (a.has_shared ? 1 : 0);
    auto group_of = [&](int slot) { return a.has_shared ? (slot == 0 ? a.E : slot - 1) : slot; };
    auto rows_of = [&](int g) { return g == a.E ? a.T : cnt_s[g]; };
    auto mblk1_of = [&](int g) {
        const int r = rows_of(g);
        return a.direct ? (r > 0 ? 1 : 0) : (r + a.tile_rows - 1) >> a.tile_shift;
    };
    // tiles per group, then an exclusive scan over the (at most 129) groups by warp 0
    const int n1_routed = a.n1_routed_blocks, n1_shared = a.n1_shared_blocks, n2 = a.n2_blocks;
    const int tmask = a.tile_rows - 1;            // tile_rows is 128 or 256
    int st_touched = 0, st_rows_r = 0, st_rows_s = 0;     // this thread's share of the call's statistics
    for (int sidx = threadIdx.x; sidx < groups; sidx += blockDim.x) {
        const int g = group_of(sidx);
        const int mblk = (rows_of(g) + a.tile_rows - 1) >> a.tile_shift;
        if (g != a.E && rows_of(g) > 0) ++st_touched;
        if (!a.direct) {
            const int r = rows_of(g), rem = r & tmask;
            const int small = a.tile_rows / 2;          // a last block of at most half a tile runs at half height
            const int run = (r & ~tmask) + (rem == 0 ? 0 : (rem <= small ? small : a.tile_rows));
            if (g == a.E) st_rows_s += run; else st_rows_r += run;
        }
        sm.pre1[sidx] = mblk1_of(g) * (g == a.E ? n1_shared : n1_routed);
        sm.pre2[sidx] = mblk * n2 * (g == a.E ? a.ksplit_shared : a.ksplit_routed);
    }
    if (rank == 0 && a.stats && threadIdx.x < ((groups + 31) & ~31)) {     // the warps that saw a group: one atomic each per counter
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            st_touched += __shfl_xor_sync(0xffffffffu, st_touched, o);
            st_rows_r += __shfl_xor_sync(0xffffffffu, st_rows_r, o);
            st_rows_s += __shfl_xor_sync(0xffffffffu, st_rows_s, o);
        }
        if ((threadIdx.x & 31) == 0) {
            if (st_touched) atomicAdd(a.stats, st_touched);
            if (st_rows_r) atomicAdd(a.stats + 1, st_rows_r);
            if (st_rows_s) atomicAdd(a.stats + 2, st_rows_s);
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        // exclusive scan over the (at most 129) groups: every lane sums its own stretch, then adds up
        // the stretch sums of the lanes before it from shared memory (32 independent broadcast
        // loads; a chain of five shuffle rounds measured 1.5 us here, a serial walk 1.2 us)
        const int lane = threadIdx.x;
        const int per = (groups + 31) / 32;
        const int base = lane * per;
        int s1 = 0, s2 = 0;
        for (int i = 0; i < per; ++i)
            if (base + i < groups) { s1 += sm.pre1[base + i]; s2 += sm.pre2[base + i]; }
        sm.part1[lane] = s1; sm.part2[lane] = s2;
        __syncwarp();
        int r1 = 0, r2 = 0, t1 = 0, t2 = 0;
#pragma unroll 8
        for (int l = 0; l < 32; ++l) {
            const int c1 = sm.part1[l], c2 = sm.part2[l];
            r1 += l < lane ? c1 : 0; r2 += l < lane ? c2 : 0;
            t1 += c1; t2 += c2;
        }
        if (lane == 0) {
            if (t1 > a.cap1 || t2 + kMaxBalanceTiles > a.cap2) { atomicOr(a.status, kStatusBadIndex); t1 = 0; t2 = 0; }
            sm.pre1[groups] = t1; sm.pre2[groups] = t2;
        }
        for (int i = 0; i < per; ++i)
            if (base + i < groups) {
                const int c1 = sm.pre1[base + i], c2 = sm.pre2[base + i];
                sm.pre1[base + i] = r1; sm.pre2[base + i] = r2;
                r1 += c1; r2 += c2;
            }
    }
    __syncthreads();
    // Balance of list 2 (see rr2): S long shared tiles come first; if S is not a multiple of the
    // consumer count C, consumers 0..rem-1 hold one long tile more.  The next (ratio-1) rounds
    // therefore hand short tiles only to consumers rem..C-1 and null tiles to the others.
    int bal_S = 0, bal_C = 0, bal_rem = 0, bal_rows = 0;
    if (a.rr2 > 0 && a.has_shared && !a.direct && a.ksplit_shared == 1 && a.ksplit_routed == 1 &&
        a.K2_shared > a.K2_routed && sm.pre2[groups] > 0) {
        bal_S = groups > 1 ? sm.pre2[1] : sm.pre2[groups];
        bal_C = a.rr2;
        bal_rem = bal_S % bal_C;
        bal_rows = bal_rem > 0 ? a.long_over_short_m1 : 0;
        if (bal_rows * bal_rem > kMaxBalanceTiles) bal_rows = 0;
    }
    const int extra2 = bal_rows * bal_rem;
    if (rank == 0 && threadIdx.x == 0) {
        a.n_tiles[0] = sm.pre1[groups];
        a.n_tiles[1] = sm.pre2[groups] + extra2;
    }
    if (extra2 == 0) {
        // No null tiles to weave in: every thread writes a contiguous run of each list, so that the
        // search for the group and the divisions are paid once per run and the rest is counting up.
        const int n_threads = n_blocks * blockDim.x, gid = rank * blockDim.x + threadIdx.x;
        for (int phase = 0; phase < 2; ++phase) {
            const int32_t *pre = phase == 0 ? sm.pre1 : sm.pre2;
            const int total = pre[groups];
            const int per = (total + n_threads - 1) / n_threads;
            const int i0 = min(gid * per, total), i1 = min(i0 + per, total);
            if (i0 >= i1) continue;
            int lo = 0, hi = groups - 1;
            while (lo < hi) {                     // last slot with pre[slot] <= i0
                const int mid = (lo + hi + 1) >> 1;
                if (pre[mid] <= i0) lo = mid; else hi = mid - 1;
            }
            int slot = lo, local = i0 - pre[lo], gsz = pre[lo + 1] - pre[lo];
            int cur = -1, g = 0, rows = 0, first = 0, m = 0, n = 0, sl = 0;
            int nn = 1, ks = 1, kchunk = 0, K = 0;     // feature blocks, K slabs, slab length, K of the group
            for (int idx = i0; idx < i1; ++idx, ++local) {
                while (local >= gsz) { local -= gsz; ++slot; gsz = pre[slot + 1] - pre[slot]; }
                if (slot != cur) {                // first tile of the run, or a new group: divide once
                    cur = slot;
                    g = group_of(slot);
                    rows = rows_of(g);
                    first = g == a.E ? 0 : off_s[g];
                    if (phase == 0) {
                        nn = g == a.E ? n1_shared : n1_routed;
                        m = local / nn; n = local - m * nn;
                    } else {
                        nn = n2;
                        ks = g == a.E ? a.ksplit_shared : a.ksplit_routed;
                        kchunk = g == a.E ? a.kchunk_shared : a.kchunk_routed;
                        K = g == a.E ? a.K2_shared : a.K2_routed;
                        m = local / (nn * ks);
                        const int rem = local - m * (nn * ks);
                        n = rem / ks; sl = rem - n * ks;
                    }
                }
                Tile t;
                t.group = g;
                if (phase == 0) {
                    if (a.direct) {
                        t.row0 = 0;
                        t.rows = a.T;
                    } else {
                        t.row0 = first + m * a.tile_rows;
                        t.rows = min(a.tile_rows, rows - m * a.tile_rows);
                    }
                    t.n0 = n * a.feat1;
                    t.k0 = 0; t.klen = a.K1; t.slot = 0;
                    t.pad = (a.tile_rows > kTileRows && t.rows <= kTileRows) ? 1 : 0;
                    a.tiles1[idx] = t;
                    if (++n == nn) { n = 0; ++m; }
                } else {
                    t.row0 = first + m * a.tile_rows;
                    t.rows = min(a.tile_rows, rows - m * a.tile_rows);
                    t.n0 = n * a.bn2;
                    t.k0 = sl * kchunk;
                    t.klen = max(0, min(kchunk, K - sl * kchunk));
                    t.slot = sl;
                    t.pad = (a.tile_rows > kTileRows && t.rows <= kTileRows) ? 1 : 0;
                    a.tiles2[idx] = t;
                    if (++sl == ks) { sl = 0; if (++n == nn) { n = 0; ++m; } }
                }
            }
        }
        return;
    }
    for (int phase = 0; phase < 2; ++phase) {
        const int32_t *pre = phase == 0 ? sm.pre1 : sm.pre2;
        const int logical = pre[groups];
        const int total = logical + (phase == 1 ? extra2 : 0);
        for (int idx = rank * blockDim.x + threadIdx.x; idx < total; idx += n_blocks * blockDim.x) {
            int i = idx;
            if (phase == 1 && extra2 > 0 && idx >= bal_S) {
                const int j = idx - bal_S;
                int shorts;
                bool null_tile = false;
                if (j < bal_rows * bal_C) {
                    const int qrow = j / bal_C, r = j % bal_C;
                    null_tile = r >= bal_C - bal_rem;
                    shorts = j - (qrow * bal_rem + max(0, r - (bal_C - bal_rem)));
                } else {
                    shorts = j - extra2;
                }
                i = bal_S + shorts;
                if (null_tile || i >= logical) {
                    Tile z;
                    z.group = 0; z.row0 = 0; z.rows = 0; z.n0 = 0; z.k0 = 0; z.klen = 0; z.slot = 0; z.pad = 0;
                    a.tiles2[idx] = z;
                    continue;
                }
            }
            int lo = 0, hi = groups - 1;
            while (lo < hi) {                     // last slot with pre[slot] <= i
                const int mid = (lo + hi + 1) >> 1;
                if (pre[mid] <= i) lo = mid; else hi = mid - 1;
            }
            const int g = group_of(lo);
            const int local = i - pre[lo];
            const int rows = rows_of(g);
            const int first = g == a.E ? 0 : off_s[g];
            Tile t;
            t.group = g; t.pad = 0;
            if (phase == 0) {
                const int n1 = g == a.E ? n1_shared : n1_routed;
                const int m = local / n1, n = local % n1;
                if (a.direct) {
                    t.row0 = 0;
                    t.rows = a.T;
                } else {
                    t.row0 = first + m * a.tile_rows;
                    t.rows = min(a.tile_rows, rows - m * a.tile_rows);
                }
                t.n0 = n * a.feat1;
                t.k0 = 0; t.klen = a.K1; t.slot = 0;
                // pair mode: a last block of at most 128 rows is marked so that the pair runs it as a
                // 128-row MMA (64 rows per CTA) instead of a 256-row one
                t.pad = (a.tile_rows > kTileRows && t.rows <= kTileRows) ? 1 : 0;
                a.tiles1[idx] = t;
            } else {
                const int ks = g == a.E ? a.ksplit_shared : a.ksplit_routed;
                const int kchunk = g == a.E ? a.kchunk_shared : a.kchunk_routed;
                const int K = g == a.E ? a.K2_shared : a.K2_routed;
                const int m = local / (n2 * ks), rem = local % (n2 * ks);
                const int n = rem / ks, sl = rem % ks;
                t.row0 = first + m * a.tile_rows;
                t.rows = min(a.tile_rows, rows - m * a.tile_rows);
                t.n0 = n * a.bn2;
                t.k0 = sl * kchunk;
                t.klen = max(0, min(kchunk, K - sl * kchunk));
                t.slot = sl;
                t.pad = (a.tile_rows > kTileRows && t.rows <= kTileRows) ? 1 : 0;
                a.tiles2[idx] = t;
            }
        }
    }
}

}  // namespace lexi
