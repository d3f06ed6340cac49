// Expert FFNs on the 5th-generation tensor cores: grouped GEMMs with tcgen05.mma, accumulators
// in tensor memory (TMEM), operands staged in shared memory by TMA (no multicast anywhere).
// Paper, Section 2: the experts E_i of y = sum G_i E_i(x); E(x) = W_down (silu(W_gate x) * (W_up x)).
//
// One persistent kernel template serves both GEMM phases and both schedules:
//   phase 1   D[token, n] = x_perm[token, :] . [W_gate; W_up][n, :]   -> h = silu(gate) * up
//   phase 2   D[token, c] = h[token, :] . W_down[c, :]                -> o (optionally split along K)
// A tile is 128 token rows (UMMA M = 128; the rows beyond a group's count are never stored) by
// BN weight rows (UMMA N), reduced over K in chunks of 64 bf16 (one 128-byte swizzle row).
//   warp 0      TMA producer (one lane)            full/empty mbarrier ring of STAGES stages
//   warp 1      TMEM allocation + MMA issue (one lane), tcgen05.commit frees stages / hands over TMEM
//   warps 2-5   epilogue: tcgen05.ld of the finished accumulator (two TMEM buffers, so the next
//               tile's MMAs overlap), SwiGLU or plain store
// Decode schedule: BN = 128, small activation box (32/64/128 rows), K split into slabs so that
// enough CTAs stream disjoint weight slices to saturate HBM; two CTAs per SM.
// Prefill schedule: BN = 256, four 48 KB stages, one CTA per SM, all 512 TMEM columns; from 128 rows
// per expert on, the CTA-pair kernel below (256-row tiles shared by a cluster of two CTAs through
// tcgen05.mma.cta_group::2, six 32 KB stages per CTA, leftover blocks as half-height tiles).
// Small decode calls read x itself in phase 1 and place rows through a position table; phase 2
// requests the weights of its first stages before it waits for phase 1 (launches are chained).
//
// Every mbarrier wait is bounded in time; a wait that runs out sets the status word and the CTA
// leaves through the common exit (TMEM is always freed).
#include <cuda.h>

#include <cstdlib>

#include <atomic>

#include "ffn_tc.h"
#include "tc_ptx.cuh"
#include "tile_build.cuh"

namespace lexi {
namespace {

using namespace tc;

struct TcParams {
    const Tile *tiles;
    const int32_t *n_tiles;      // device: number of tiles in the list
    int32_t E;                   // group == E is the shared expert
    int32_t N_routed, N_shared;  // row pitch and column bound of the outputs
    void *out_routed, *out_shared;
    unsigned long long slab_stride_routed, slab_stride_shared;   // elements between split-K slabs
    int32_t *status;
    const int32_t *pos;          // direct mode: pos[group * pos_stride + token] = output row or -1
    int32_t pos_stride;
    const int32_t *row_map;      // not null: routed output row r goes to row row_map[r] (0 <= row_map[r] < row_map_n)
    int32_t row_map_n;
};

// Where routed output row `row` is stored: itself, or its entry of the row map; an entry outside
// the buffer raises the bad-index status and the row is dropped (-1).
__device__ __forceinline__ int mapped_row(const TcParams &p, int row) {
    if (p.row_map == nullptr) return row;
    const int v = p.row_map[row];
    if ((unsigned)v >= (unsigned)p.row_map_n) { atomicOr(p.status, kStatusBadIndex); return -1; }
    return v;
}

// Phase-2 tiles of the prefill schedule pass their fp32 output through a per-warp staging buffer
// (32 rows x 32 columns, row pitch 36 floats) so that global stores are row-contiguous.
constexpr int kStagePitch = 36;
constexpr int kStageBytes = 4 * 32 * kStagePitch * 4;

template <int PHASE, int BN, typename OutT>
__host__ __device__ constexpr bool tc_staged_out() { return PHASE == 2 && BN == 256 && sizeof(OutT) == 4; }

template <int A_ROWS, int BN, int STAGES>
constexpr int tc_smem_bytes(bool staged) {
    return STAGES * (A_ROWS * 128 + BN * 128) + 1024 /* alignment slack */ + 256 /* barriers */ +
           (staged ? kStageBytes : 0);
}

__device__ __forceinline__ float silu_mul(float g, float u) {
    return __fdividef(g, 1.0f + __expf(-g)) * u;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <int PHASE, int BN, int A_ROWS, int STAGES, int MIN_CTAS, typename OutT>
__global__ void __launch_bounds__(192, MIN_CTAS)
ffn_tc_kernel(const __grid_constant__ CUtensorMap mapA_routed, const __grid_constant__ CUtensorMap mapA_shared,
              const __grid_constant__ CUtensorMap mapB0_routed, const __grid_constant__ CUtensorMap mapB1_routed,
              const __grid_constant__ CUtensorMap mapB0_shared, const __grid_constant__ CUtensorMap mapB1_shared,
              const TcParams p) {
    constexpr int A_BYTES = A_ROWS * 128;
    constexpr int B_BYTES = BN * 128;
    constexpr int TMEM_COLS = 2 * BN;
    static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "TMEM columns: power of two");
    static_assert(STAGES * B_BYTES >= 128 * 128, "the 128-row operand read must stay inside the allocation");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t a_base = base;
    const uint32_t b_base = base + STAGES * A_BYTES;
    const uint32_t bar_base = b_base + STAGES * B_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    const uint32_t slot_addr = bar_base + 8u * (2 * STAGES + 4);
    volatile uint32_t *slot_ptr = reinterpret_cast<volatile uint32_t *>(smem_raw + (slot_addr - raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        tma_prefetch_map(&mapA_routed); tma_prefetch_map(&mapA_shared);
        tma_prefetch_map(&mapB0_routed); tma_prefetch_map(&mapB0_shared);
        if (PHASE == 1) { tma_prefetch_map(&mapB1_routed); tma_prefetch_map(&mapB1_shared); }
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 128); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(slot_addr, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *slot_ptr;
    // Phase 2 only: the tile lists were finished two kernels ago (phase 1 lets its successor start
    // only after its own wait), and weights never change, so the weight halves of the first stages
    // of this CTA's first tile are requested before waiting for phase 1; h follows after the wait.
    int preloaded = 0;
    if (PHASE == 2 && threadIdx.x == 0) {
        const int nt = *p.n_tiles;
        if ((int)blockIdx.x < nt) {
            const Tile t = p.tiles[blockIdx.x];
            const bool shared = t.group == p.E;
            const int nk = (t.klen + kBK - 1) / kBK;
            preloaded = nk < STAGES ? nk : STAGES;
            for (int kc = 0; kc < preloaded; ++kc) {
                mbar_expect_tx(full_bar(kc), A_BYTES + B_BYTES);
                tma_load_3d(b_base + kc * B_BYTES, shared ? &mapB0_shared : &mapB0_routed, full_bar(kc),
                            t.k0 + kc * kBK, t.n0, shared ? 0 : t.group);
            }
        }
    }
    // everything above overlaps the tail of the previous kernel; its results are needed from here on
    pdl_wait();
    pdl_trigger();
    // the tile count and this CTA's first tile record are independent loads (the record lies inside
    // the list's allocation whether or not it is valid); every role starts from them
    const Tile first_tile = p.tiles[blockIdx.x];
    const int n_tiles = *p.n_tiles;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            Tile t_next = first_tile;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
                const Tile t = t_next;       // the next tile's record is fetched while this one streams
                if (tile + (int)gridDim.x < n_tiles) t_next = p.tiles[tile + gridDim.x];
                const bool shared = t.group == p.E;
                const CUtensorMap *mA = shared ? &mapA_shared : &mapA_routed;
                const CUtensorMap *mB0 = shared ? &mapB0_shared : &mapB0_routed;
                const CUtensorMap *mB1 = shared ? &mapB1_shared : &mapB1_routed;
                const int grp = shared ? 0 : t.group;
                const int nk = (t.klen + kBK - 1) / kBK;
                for (int kc = 0; kc < nk; ++kc, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    const int k = t.k0 + kc * kBK;
                    if (PHASE == 2 && (int)it < preloaded) {     // weights of this stage are already on their way
                        tma_load_3d(a_base + s * A_BYTES, mA, full_bar(s), k, t.row0, 0);
                        continue;
                    }
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, p.status)) { ok = false; break; }
                    mbar_expect_tx(full_bar(s), A_BYTES + B_BYTES);
                    tma_load_3d(a_base + s * A_BYTES, mA, full_bar(s), k, t.row0, 0);
                    if (PHASE == 1) {
                        tma_load_3d(b_base + s * B_BYTES, mB0, full_bar(s), k, t.n0, grp);
                        tma_load_3d(b_base + s * B_BYTES + B_BYTES / 2, mB1, full_bar(s), k, t.n0, grp);
                    } else {
                        tma_load_3d(b_base + s * B_BYTES, mB0, full_bar(s), k, t.n0, grp);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // tiles of at most 64 rows run as M = 64 MMAs (half the tensor-core time); their 64 rows
            // sit in lanes 0-15 of each 32-lane quarter of TMEM
            constexpr uint32_t idesc128 = make_idesc_bf16(BN), idesc64 = make_idesc_bf16_m(64, BN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            Tile t_nx = first_tile;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++tcount) {
                const int nk = (t_nx.klen + kBK - 1) / kBK;
                const uint32_t idesc = t_nx.rows <= 64 ? idesc64 : idesc128;
                if (tile + (int)gridDim.x < n_tiles) t_nx = p.tiles[tile + gridDim.x];
                const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), bph ^ 1u, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kc = 0; kc < nk; ++kc, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(full_bar(s), ph, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_kmajor_sw128_desc(a_base + s * A_BYTES);
                    const uint64_t b_desc = make_kmajor_sw128_desc(b_base + s * B_BYTES);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk)     // 32 bytes along K per instruction
                        umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kc | kk) != 0);
                    umma_commit(empty_bar(s));
                }
                if (ok) umma_commit(tfull_bar(buf));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                  // TMEM lane quarter this warp may read
        uint32_t tcount = 0;
        Tile t_next = first_tile;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tcount) {
            const Tile t = t_next;
            if (tile + (int)gridDim.x < n_tiles) t_next = p.tiles[tile + gridDim.x];
            const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
            // everything that depends only on the tile record comes before the wait for its accumulator
            const bool shared = t.group == p.E;
            const int N = shared ? p.N_shared : p.N_routed;
            // M = 128: lane = row.  M = 64 (rows <= 64): row 16 q + l lives in lane l < 16 of quarter q.
            const bool small = t.rows <= 64;
            const int row_in_tile = small ? (lane < 16 ? q * 16 + lane : 1 << 20) : q * 32 + lane;
            bool row_ok = row_in_tile < t.rows;
            int out_row = t.row0 + row_in_tile;
            if (p.pos != nullptr && !shared) {   // direct mode: the tile holds all tokens, keep the routed ones
                out_row = row_ok ? p.pos[t.group * p.pos_stride + row_in_tile] : -1;
                row_ok = out_row >= 0;
            }
            if (PHASE == 2 && p.row_map != nullptr && !shared && row_ok) {
                out_row = mapped_row(p, out_row);
                row_ok = out_row >= 0;
            }
            const bool got = mbar_wait(tfull_bar(buf), bph, p.status);
            if (!__all_sync(0xffffffffu, got)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN;
            OutT *out = reinterpret_cast<OutT *>(shared ? p.out_shared : p.out_routed) +
                        (size_t)t.slot * (shared ? p.slab_stride_shared : p.slab_stride_routed) +
                        (size_t)(row_ok ? out_row : 0) * N + t.n0;
            if (PHASE == 1) {
#pragma unroll 1
                for (int c = 0; c < BN / 2; c += 16) {
                    uint32_t g[16], u[16];
                    tmem_ld16(taddr + c, g);
                    tmem_ld16(taddr + BN / 2 + c, u);
                    tmem_ld_wait();
                    uint32_t packed[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        packed[i] = pack_bf16(silu_mul(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                                              silu_mul(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
                    if (row_ok) {
                        if (t.n0 + c + 8 <= N)
                            *reinterpret_cast<uint4 *>(out + c) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                        if (t.n0 + c + 16 <= N)
                            *reinterpret_cast<uint4 *>(out + c + 8) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
                    }
                }
            } else if constexpr (tc_staged_out<PHASE, BN, OutT>()) {
                // each lane parks its row's 32 columns in shared memory; the warp then writes them
                // out four rows per instruction, 128 contiguous bytes per row
                float *stg = reinterpret_cast<float *>(smem_raw + (bar_base + 256u - raw)) + q * 32 * kStagePitch;
                const int warp_row0 = small ? q * 16 : q * 32;        // first tile row held by this warp
                OutT *wbase = reinterpret_cast<OutT *>(shared ? p.out_shared : p.out_routed) +
                              (size_t)t.slot * (shared ? p.slab_stride_shared : p.slab_stride_routed) +
                              (size_t)(t.row0 + warp_row0) * N + t.n0;
                const int rows_here = min(t.rows - warp_row0, small ? 16 : 32);   // valid rows of this warp
                const int rr0 = lane >> 3, cc = 4 * (lane & 7);
                long long drow[8];                 // destination of the eight rows this lane stores, relative to wbase
                uint32_t row_mask = 0;             // bit j: row 4 j + rr0 exists and has a destination
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int rr = 4 * j + rr0;
                    bool ok_row = rr < rows_here;
                    drow[j] = rr;
                    if (p.row_map != nullptr && !shared && ok_row) {
                        const int m = mapped_row(p, t.row0 + warp_row0 + rr);
                        ok_row = m >= 0;
                        drow[j] = (long long)m - (t.row0 + warp_row0);
                    }
                    row_mask |= (ok_row ? 1u : 0u) << j;
                }
#pragma unroll 1
                for (int c = 0; c < BN; c += 32) {
                    uint32_t v0[16], v1[16];
                    tmem_ld16(taddr + c, v0);
                    tmem_ld16(taddr + c + 16, v1);
                    tmem_ld_wait();
                    uint4 *wr = reinterpret_cast<uint4 *>(stg + lane * kStagePitch);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        wr[i] = make_uint4(v0[4 * i], v0[4 * i + 1], v0[4 * i + 2], v0[4 * i + 3]);
                        wr[4 + i] = make_uint4(v1[4 * i], v1[4 * i + 1], v1[4 * i + 2], v1[4 * i + 3]);
                    }
                    __syncwarp();
                    const bool col_ok = t.n0 + c + cc + 4 <= N;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int rr = 4 * j + rr0;
                        const uint4 val = *reinterpret_cast<const uint4 *>(stg + rr * kStagePitch + cc);
                        if (((row_mask >> j) & 1u) && col_ok)
                            *reinterpret_cast<uint4 *>(wbase + drow[j] * N + c + cc) = val;
                    }
                    __syncwarp();
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < BN; c += 16) {
                    uint32_t v[16];
                    tmem_ld16(taddr + c, v);
                    tmem_ld_wait();
                    if (row_ok) {
                        if (sizeof(OutT) == 4) {
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                if (t.n0 + c + 4 * i + 4 <= N)
                                    *reinterpret_cast<uint4 *>(out + c + 4 * i) =
                                        make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 2; ++i)
                                if (t.n0 + c + 8 * i + 8 <= N)
                                    *reinterpret_cast<uint4 *>(out + c + 8 * i) = make_uint4(
                                        pack_bf16(__uint_as_float(v[8 * i]), __uint_as_float(v[8 * i + 1])),
                                        pack_bf16(__uint_as_float(v[8 * i + 2]), __uint_as_float(v[8 * i + 3])),
                                        pack_bf16(__uint_as_float(v[8 * i + 4]), __uint_as_float(v[8 * i + 5])),
                                        pack_bf16(__uint_as_float(v[8 * i + 6]), __uint_as_float(v[8 * i + 7])));
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(buf));
        }
    }

    // ---------------------------------------------------------------- common exit
    __syncwarp();
    if (*reinterpret_cast<volatile int32_t *>(p.status) & kStatusTimeout) {
        // a wait ran out somewhere: give copies and MMAs still in flight time to land before the
        // shared memory and TMEM of this CTA are handed back
        for (int i = 0; i < 256; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------ CTA-pair variant (prefill)
// Tile = 256 token rows x 256 weight rows, worked on by the two CTAs of a cluster of 2 with
// tcgen05.mma.cta_group::2: CTA r holds rows 128r..128r+127 of the tile (A and D) and half of B
// (phase 1: CTA 0 the 128 gate rows, CTA 1 the 128 up rows; phase 2: 128 rows of W_down each), so a
// stage costs 32 KB of loads per CTA instead of 48 KB.  CTA 0 issues all MMAs once both CTAs' loads
// have landed (both count their bytes on CTA 0's "full" mbarrier); tcgen05.commit multicasts the
// "stage free" and "accumulator ready" arrivals to both CTAs; both epilogues release the accumulator
// on CTA 0's "empty" mbarrier.  No multicast loads.  Waits are bounded as in the 1-CTA kernel.
constexpr int kPairStages = 6;
constexpr int kPairABytes = 128 * 128, kPairBBytes = 128 * 128;

template <int PHASE>
constexpr int pair_smem_bytes() {
    return kPairStages * (kPairABytes + kPairBBytes) + 1024 + 256 + (PHASE == 2 ? kStageBytes : 0);
}

template <int PHASE, typename OutT>
__global__ void __launch_bounds__(192, 1)
ffn_tc_pair_kernel(const __grid_constant__ CUtensorMap mapA_routed, const __grid_constant__ CUtensorMap mapA_shared,
                   const __grid_constant__ CUtensorMap mapB0_routed, const __grid_constant__ CUtensorMap mapB1_routed,
                   const __grid_constant__ CUtensorMap mapB0_shared, const __grid_constant__ CUtensorMap mapB1_shared,
                   const __grid_constant__ CUtensorMap mapG64_routed, const __grid_constant__ CUtensorMap mapU64_routed,
                   const __grid_constant__ CUtensorMap mapG64_shared, const __grid_constant__ CUtensorMap mapU64_shared,
                   const TcParams p) {
    // Half-height tiles (Tile::pad = 1, at most 128 valid rows): the pair issues M = 128 MMAs, 64 rows
    // per CTA.  Then each CTA's accumulator holds its 64 rows twice over the lanes: lanes 0-63 carry
    // output columns 0-127 (B rows of CTA 0), lanes 64-127 columns 128-255 (B rows of CTA 1), both in
    // TMEM columns 0-127.  Phase 1 therefore gives each CTA 64 gate rows followed by 64 up rows of the
    // same 64 features (mapG64/mapU64, 64-row boxes), so that gate and up of a feature meet in a thread.
    constexpr int BN = 256, STAGES = kPairStages, A_BYTES = kPairABytes, B_BYTES = kPairBBytes;
    constexpr int TMEM_COLS = 2 * BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t a_base = base;
    const uint32_t b_base = base + STAGES * A_BYTES;
    const uint32_t bar_base = b_base + STAGES * B_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    const uint32_t slot_addr = bar_base + 8u * (2 * STAGES + 4);
    volatile uint32_t *slot_ptr = reinterpret_cast<volatile uint32_t *>(smem_raw + (slot_addr - raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0: issues the MMAs
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 256); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(slot_addr, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem_base = *slot_ptr;
    pdl_wait();
    pdl_trigger();
    const int n_tiles = *p.n_tiles;
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one lane, both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            Tile t_next = pair_id < n_tiles ? p.tiles[pair_id] : Tile{};
            for (int tile = pair_id; ok && tile < n_tiles; tile += n_pairs) {
                const Tile t = t_next;
                if (tile + n_pairs < n_tiles) t_next = p.tiles[tile + n_pairs];
                const bool shared = t.group == p.E;
                const bool half = t.pad != 0;
                const CUtensorMap *mA = shared ? &mapA_shared : &mapA_routed;
                // this CTA's half of B: phase 1 -> gate rows (CTA 0) or up rows (CTA 1) of the same
                // features; phase 2 -> rows n0 + 128 rank of W_down
                const CUtensorMap *mB = PHASE == 1 ? (rank == 0 ? (shared ? &mapB0_shared : &mapB0_routed)
                                                                : (shared ? &mapB1_shared : &mapB1_routed))
                                                   : (shared ? &mapB0_shared : &mapB0_routed);
                const int b_row = PHASE == 1 ? t.n0 : t.n0 + 128 * (int)rank;
                const int grp = shared ? 0 : t.group;
                const int a_row = t.row0 + (half ? 64 : 128) * (int)rank;
                const int nk = (t.klen + kBK - 1) / kBK;
                for (int kc = 0; kc < nk; ++kc, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, p.status)) { ok = false; break; }
                    const uint32_t full0 = full_bar(s) & kPeerBitMask;      // CTA 0 counts both CTAs' bytes
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2 * (A_BYTES + B_BYTES));
                    const int k = t.k0 + kc * kBK;
                    tma_load_3d_pair(a_base + s * A_BYTES, mA, full0, k, a_row, 0);
                    if (PHASE == 1 && half) {
                        const int f = t.n0 + 64 * (int)rank;      // this CTA's 64 features: gate rows, then up rows
                        tma_load_3d_pair(b_base + s * B_BYTES, shared ? &mapG64_shared : &mapG64_routed, full0, k, f, grp);
                        tma_load_3d_pair(b_base + s * B_BYTES + B_BYTES / 2, shared ? &mapU64_shared : &mapU64_routed,
                                         full0, k, f, grp);
                    } else {
                        tma_load_3d_pair(b_base + s * B_BYTES, mB, full0, k, b_row, grp);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (CTA 0 only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc_full = make_idesc_bf16_m(256, BN), idesc_half = make_idesc_bf16_m(128, BN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            Tile t_next = pair_id < n_tiles ? p.tiles[pair_id] : Tile{};
            for (int tile = pair_id; ok && tile < n_tiles; tile += n_pairs, ++tcount) {
                const int nk = (t_next.klen + kBK - 1) / kBK;
                const uint32_t idesc = t_next.pad ? idesc_half : idesc_full;
                if (tile + n_pairs < n_tiles) t_next = p.tiles[tile + n_pairs];
                const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), bph ^ 1u, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kc = 0; kc < nk; ++kc, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(full_bar(s), ph, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_kmajor_sw128_desc(a_base + s * A_BYTES);
                    const uint64_t b_desc = make_kmajor_sw128_desc(b_base + s * B_BYTES);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk)
                        umma_bf16_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kc | kk) != 0);
                    umma_commit_pair(empty_bar(s));
                }
                if (ok) umma_commit_pair(tfull_bar(buf));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int q = warp & 3;
        const int row_in_cta = q * 32 + lane;                    // TMEM lane of this thread
        uint32_t tcount = 0;
        Tile t_next = pair_id < n_tiles ? p.tiles[pair_id] : Tile{};
        for (int tile = pair_id; tile < n_tiles; tile += n_pairs, ++tcount) {
            const Tile t = t_next;
            if (tile + n_pairs < n_tiles) t_next = p.tiles[tile + n_pairs];
            const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
            const bool shared = t.group == p.E;
            const bool half = t.pad != 0;
            const int N = shared ? p.N_shared : p.N_routed;
            // full tile: lane = row of this CTA's 128, all 256 columns.  Half tile: lane % 64 = row of
            // this CTA's 64, lane / 64 picks output columns 0-127 or 128-255 (TMEM columns 0-127 both).
            const int cb = half ? (row_in_cta >> 6) : 0;
            const int row_in_tile = half ? 64 * (int)rank + (row_in_cta & 63) : 128 * (int)rank + row_in_cta;
            const bool row_ok = row_in_tile < t.rows;
            const bool got = mbar_wait(tfull_bar(buf), bph, p.status);
            if (!__all_sync(0xffffffffu, got)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN;
            OutT *obase = reinterpret_cast<OutT *>(shared ? p.out_shared : p.out_routed) +
                          (size_t)t.slot * (shared ? p.slab_stride_shared : p.slab_stride_routed);
            if (PHASE == 1) {
                const int feats = half ? 64 : 128;               // features this thread finishes
                const int f0 = t.n0 + 64 * cb;
                OutT *out = obase + (size_t)(t.row0 + row_in_tile) * N + f0;
#pragma unroll 1
                for (int c = 0; c < feats; c += 16) {
                    uint32_t g[16], u[16];
                    tmem_ld16(taddr + c, g);
                    tmem_ld16(taddr + feats + c, u);
                    tmem_ld_wait();
                    uint32_t packed[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        packed[i] = pack_bf16(silu_mul(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                                              silu_mul(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
                    if (row_ok) {
                        if (f0 + c + 8 <= N)
                            *reinterpret_cast<uint4 *>(out + c) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                        if (f0 + c + 16 <= N)
                            *reinterpret_cast<uint4 *>(out + c + 8) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
                    }
                }
            } else {
                // this warp's 32 rows of the tile and its first output column; the accumulator is read
                // in fragment layout (16 lanes x 64 columns at a time) and stored straight from the
                // registers: four threads fill a 32-byte sector, and no shared memory is touched,
                // which the MMA operand reads and the TMA writes already keep busy
                const int warp_row0 = half ? 64 * (int)rank + 32 * (q & 1) : 128 * (int)rank + 32 * q;
                const int col0 = t.n0 + (half ? 128 * (q >> 1) : 0);
                const int cols = half ? 128 : BN;
                OutT *wbase = obase + (size_t)(t.row0 + warp_row0) * N + col0;
                const int rows_here = t.rows - warp_row0;
                static_assert(PHASE != 2 || sizeof(OutT) == 4, "the down projection's outputs are fp32");
                const int fr = lane >> 2, fc = 2 * (lane & 3);
#pragma unroll 1
                for (int hl = 0; hl < 2; ++hl) {
                    const int ra = 16 * hl + fr, rb = ra + 8;
                    bool oka = ra < rows_here, okb = rb < rows_here;
                    long long da = ra, db = rb;            // destination rows relative to wbase
                    if (p.row_map != nullptr && !shared) {
                        const int first = t.row0 + warp_row0;
                        const int ma = oka ? mapped_row(p, first + ra) : -1, mb = okb ? mapped_row(p, first + rb) : -1;
                        oka = ma >= 0; okb = mb >= 0;
                        da = (long long)ma - first; db = (long long)mb - first;
                    }
                    OutT *pa = wbase + da * N + fc, *pb = wbase + db * N + fc;
#pragma unroll 1
                    for (int c = 0; c < cols; c += 64) {
                        uint32_t v[32];
                        tmem_ld_16x256b_x8(taddr + ((uint32_t)(16 * hl) << 16) + c, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int col = c + 8 * j;
                            if (col0 + col + fc + 2 <= N) {
                                if (oka) *reinterpret_cast<uint2 *>(pa + col) = make_uint2(v[4 * j], v[4 * j + 1]);
                                if (okb) *reinterpret_cast<uint2 *>(pb + col) = make_uint2(v[4 * j + 2], v[4 * j + 3]);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive_cta0(tempty_bar(buf));       // both CTAs' epilogues free the buffer on CTA 0
        }
    }

    // ---------------------------------------------------------------- common exit
    __syncwarp();
    if (*reinterpret_cast<volatile int32_t *>(p.status) & kStatusTimeout) {
        for (int i = 0; i < 256; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // neither CTA leaves while the other may still reach into it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// One thread waits on an mbarrier that nothing will ever arrive on, with a short limit: the same
// bounded wait as in the GEMM kernels, used by the test of the time-out path.
__global__ void wait_probe_kernel(int32_t *status, unsigned long long limit_ns) {
    __shared__ unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(b, 0, status, limit_ns);
    }
}

// ------------------------------------------------------------------ tile lists
__global__ void __launch_bounds__(1024) build_tiles_kernel(TileBuildArgs a) {
    pdl_trigger();
    pdl_wait();
    __shared__ TileBuildSmem sm;
    __shared__ int32_t cnt_s[kMaxExperts + 1], off_s[kMaxExperts + 1];
    for (int e = threadIdx.x; e < a.E; e += blockDim.x) { cnt_s[e] = a.counts[e]; off_s[e] = a.offsets[e]; }
    __syncthreads();
    build_tiles_block(a, cnt_s, off_s, sm);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                             CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                             CUtensorMapFloatOOBfill);

// bf16 tensor [groups, rows, K] (K contiguous), box = 64 x box_rows x 1, 128-byte swizzle,
// out-of-range elements read as zero.
bool encode_map(const TcState *st, CUtensorMap *m, const void *ptr, uint64_t K, uint64_t rows,
                uint64_t groups, uint32_t box_rows) {
    cuuint64_t dims[3] = {K, rows, groups};
    cuuint64_t strides[2] = {K * 2, rows * K * 2};
    cuuint32_t box[3] = {(cuuint32_t)kBK, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = reinterpret_cast<EncodeFn>(st->encode_fn)(
        m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int ceil_div(int a, int b) { return (a + b - 1) / b; }
int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }
int slabs_for(int K) { return clampi(ceil_div(K, 1024), 1, 8); }
size_t decode_row_cap(const moe_config_t &c) {
    const size_t pairs = (size_t)c.max_T * c.max_k;
    const size_t cap = (size_t)16 * c.E;
    return pairs < cap ? pairs : cap;
}

constexpr int kMaxTcDevices = 64;
int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxTcDevices) { cudaGetLastError(); return -1; }
    return dev;
}

template <int PHASE, int BN, int A_ROWS, int STAGES, int MIN_CTAS, typename OutT>
cudaError_t launch_tc(const CUtensorMap *maps, const TcParams &p, int grid, cudaStream_t s, bool chained) {
    auto kern = ffn_tc_kernel<PHASE, BN, A_ROWS, STAGES, MIN_CTAS, OutT>;
    constexpr int smem = tc_smem_bytes<A_ROWS, BN, STAGES>(tc_staged_out<PHASE, BN, OutT>());
    // the shared-memory opt-in belongs to the kernel on one device
    static std::atomic<bool> configured[kMaxTcDevices];
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    return launch_chained(kern, dim3(grid), dim3(192), smem, s, chained,
                          maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], p);
}

template <int PHASE, typename OutT>
cudaError_t launch_tc_pair(const CUtensorMap *maps, const TcParams &p, int max_pairs, cudaStream_t s, bool chained) {
    auto kern = ffn_tc_pair_kernel<PHASE, OutT>;
    constexpr int smem = pair_smem_bytes<PHASE>();
    static std::atomic<int> max_clusters_dev[kMaxTcDevices];     // 0: not asked yet on that device
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    int max_clusters = max_clusters_dev[dev].load(std::memory_order_acquire);
    cudaLaunchConfig_t cfg{};
    cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    if (max_clusters <= 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3(2 * 74);
        cfg.numAttrs = 1;
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorInvalidConfiguration;
        max_clusters = n;
        max_clusters_dev[dev].store(n, std::memory_order_release);
    }
    const int clusters = max_pairs < max_clusters ? (max_pairs < 1 ? 1 : max_pairs) : max_clusters;
    cfg.gridDim = dim3(2 * clusters);
    cfg.numAttrs = chained ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, maps[0], maps[1], maps[2], maps[3], maps[4], maps[5],
                              maps[6], maps[7], maps[8], maps[9], p);
}

}  // namespace

bool tc_encode_bf16_map(const TcState *st, void *map, const void *ptr, uint64_t K, uint64_t rows,
                        uint64_t groups, uint32_t box_rows) {
    return st->ready && encode_map(st, reinterpret_cast<CUtensorMap *>(map), ptr, K, rows, groups, box_rows);
}

bool tc_shape_ok(const moe_config_t &c) {
    if (c.dtype != MOE_BF16) return false;
    if (c.d < 64 || c.I < 64 || (c.I_shared > 0 && c.I_shared < 64)) return false;
    return c.d % 8 == 0 && c.I % 8 == 0 && c.I_shared % 8 == 0;
}
int tc_max_slabs(const moe_config_t &c) { return slabs_for(c.I); }
int tc_max_shared_slabs(const moe_config_t &c) { return c.I_shared > 0 ? slabs_for(c.I_shared) : 1; }

size_t tc_o_elems(const moe_config_t &c, int slabs) {
    const size_t pairs = (size_t)c.max_T * c.max_k;
    const size_t full = pairs * c.d;                              // one fp32 slab for every pair
    const size_t dec = decode_row_cap(c) * (size_t)slabs * c.d;   // split-K slabs, decode-sized calls
    return full > dec ? full : dec;
}
size_t tc_os_elems(const moe_config_t &c, int slabs) {
    const size_t full = (size_t)c.max_T * c.d;
    const size_t rows = (size_t)c.max_T < (size_t)16 * c.E ? (size_t)c.max_T : (size_t)16 * c.E;
    const size_t dec = rows * (size_t)slabs * c.d;
    return full > dec ? full : dec;
}
size_t tc_max_tiles(const moe_config_t &c, int phase) {
    const size_t pairs = (size_t)c.max_T * c.max_k;
    const size_t mblk_routed = pairs / kTileRows + (pairs < (size_t)c.E ? pairs : (size_t)c.E);
    const size_t mblk_shared = c.I_shared > 0 ? ((size_t)c.max_T + kTileRows - 1) / kTileRows : 0;
    if (phase == 1)
        return mblk_routed * ceil_div(c.I, 32) + mblk_shared * ceil_div(c.I_shared > 0 ? c.I_shared : 32, 32) + 1;
    return mblk_routed * ceil_div(c.d, 64) * slabs_for(c.I) +
           mblk_shared * ceil_div(c.d, 64) * (c.I_shared > 0 ? slabs_for(c.I_shared) : 1) + 1 + kMaxBalanceTiles;
}

cudaError_t launch_wait_probe(int32_t *status, unsigned long long limit_ns, cudaStream_t s) {
    wait_probe_kernel<<<1, 32, 0, s>>>(status, limit_ns);
    return cudaGetLastError();
}

int tc_state_init(TcState *st, const moe_config_t &c) {
    if (!tc_shape_ok(c)) return MOE_OK;     // SIMT-only plan
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    st->encode_fn = fn;
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&st->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    st->ready = true;
    return MOE_OK;
}

void tc_make_schedule(const moe_config_t &c, const Workspace &ws, const FfnArgs &a, int schedule,
                      bool direct, int sm_count, TcSchedule *out) {
    const bool decode = schedule == MOE_SCHED_DECODE;
    const int rows = a.T * a.k;
    const bool has_shared = a.I_s > 0;
    TcSchedule &sc = *out;
    sc.decode = decode;
    sc.direct = direct;
    // Prefill: the GEMMs run on CTA pairs (256-row tiles, cta_group::2, leftovers as half-height
    // tiles); measured at least as fast as the 1-CTA kernel from 64 rows per expert upwards.
    // LEXI_PREFILL_2CTA=0 / =1 forces the choice.
    // Below 64 rows per expert the one-CTA 128x256 kernel measured 3-6 % faster (its tiles are half as
    // tall, and the call is bound by the weight stream rather than by the tensor cores).
    static const char *pair_env = getenv("LEXI_PREFILL_2CTA");
    const bool pair_auto = (long long)rows >= 64ll * a.E;
    sc.pair = !decode && !direct && schedule != MOE_SCHED_PREFILL_1CTA && (pair_env ? pair_env[0] == '1' : pair_auto);
    sc.bn1 = decode ? 128 : 256;          // phase-1 tile: bn1/2 gate rows + bn1/2 up rows
    sc.bn2 = decode ? 128 : 256;
    sc.a_rows = 128;
    if (decode) sc.a_rows = a.T <= 32 ? 32 : (a.T <= 64 ? 64 : 128);
    int ks_r = 1, ks_s = 1;
    if (decode && (size_t)rows <= decode_row_cap(c)) {
        ks_r = slabs_for(a.I);
        ks_s = has_shared ? slabs_for(a.I_s) : 1;
    }
    sc.kchunk_r = ceil_div(ceil_div(a.I, ks_r), kBK) * kBK;
    sc.kchunk_s = has_shared ? ceil_div(ceil_div(a.I_s, ks_s), kBK) * kBK : kBK;
    sc.ks_r = ceil_div(a.I, sc.kchunk_r);
    sc.ks_s = has_shared ? ceil_div(a.I_s, sc.kchunk_s) : 1;

    TileBuildArgs &tb = sc.tb;
    tb = TileBuildArgs{};
    tb.counts = a.counts; tb.offsets = a.offsets; tb.E = a.E; tb.T = a.T; tb.has_shared = has_shared;
    tb.feat1 = sc.bn1 / 2; tb.N1_routed = a.I; tb.N1_shared = a.I_s; tb.K1 = a.d;
    tb.bn2 = sc.bn2; tb.N2 = a.d; tb.K2_routed = a.I; tb.K2_shared = a.I_s;
    tb.ksplit_routed = sc.ks_r; tb.kchunk_routed = sc.kchunk_r;
    tb.ksplit_shared = sc.ks_s; tb.kchunk_shared = sc.kchunk_s;
    tb.tiles1 = ws.tiles1; tb.tiles2 = ws.tiles2; tb.n_tiles = ws.n_tiles;
    tb.cap1 = (int)tc_max_tiles(c, 1); tb.cap2 = (int)tc_max_tiles(c, 2);
    tb.status = ws.status;
    tb.direct = direct ? 1 : 0;
    tb.tile_rows = sc.pair ? 2 * kTileRows : kTileRows;
    tb.tile_shift = sc.pair ? 8 : 7;
    static_assert(kTileRows == 128, "tile_shift");
    tb.n1_routed_blocks = (tb.N1_routed + tb.feat1 - 1) / tb.feat1;
    tb.n1_shared_blocks = (tb.N1_shared + tb.feat1 - 1) / tb.feat1;
    tb.n2_blocks = (tb.N2 + tb.bn2 - 1) / tb.bn2;
    tb.long_over_short_m1 = tb.K2_routed > 0 ? (tb.K2_shared + tb.K2_routed - 1) / tb.K2_routed - 1 : 0;
    // prefill: consumers of the phase-2 list (CTAs, or CTA pairs), for the balance of long shared tiles
    tb.rr2 = (!decode && !direct && has_shared) ? (sc.pair ? sm_count / 2 : sm_count) : 0;
    tb.stats = ws.stats;
}

int tc_ffn_forward(TcState *st, const moe_config_t &c, const Workspace &ws, const FfnArgs &a,
                   const TcSchedule &sc, int sm_count, cudaStream_t s, uint64_t *launches,
                   TcOutputLayout *layout) {
    if (!st->ready) return MOE_ERR_SHAPE;
    const bool decode = sc.decode;
    const int rows = a.T * a.k;
    const bool has_shared = a.I_s > 0;
    const size_t pairs_alloc = (size_t)c.max_T * c.max_k;
    const int bn1 = sc.bn1, bn2 = sc.bn2, a_rows = sc.a_rows, ks_r = sc.ks_r, ks_s = sc.ks_s;

    // ---- tensor maps
    CUtensorMap m1[10], m2[10];
    bool ok = true;
    const void *dummy = a.x;   // maps of an absent shared expert are never dereferenced
    if (sc.direct) ok = ok && encode_map(st, &m1[0], a.x, a.d, a.T, 1, a_rows);   // every group reads x itself
    else ok = ok && encode_map(st, &m1[0], a.x_perm, a.d, a.x_perm_rows ? a.x_perm_rows : pairs_alloc + 128, 1, a_rows);
    ok = ok && encode_map(st, &m1[1], a.x, a.d, a.T, 1, a_rows);
    ok = ok && encode_map(st, &m1[2], a.W_gate, a.d, a.I, a.E, bn1 / 2);
    ok = ok && encode_map(st, &m1[3], a.W_up, a.d, a.I, a.E, bn1 / 2);
    ok = ok && encode_map(st, &m1[4], has_shared ? a.Ws_gate : dummy, a.d, has_shared ? a.I_s : a.T, 1, bn1 / 2);
    ok = ok && encode_map(st, &m1[5], has_shared ? a.Ws_up : dummy, a.d, has_shared ? a.I_s : a.T, 1, bn1 / 2);
    ok = ok && encode_map(st, &m2[0], a.h, a.I, pairs_alloc + 128, 1, a_rows);
    ok = ok && encode_map(st, &m2[1], has_shared ? a.h_s : a.h, has_shared ? a.I_s : a.I,
                          has_shared ? (size_t)c.max_T + 128 : pairs_alloc + 128, 1, a_rows);
    ok = ok && encode_map(st, &m2[2], a.W_down, a.I, a.d, a.E, sc.pair ? 128 : bn2);
    m2[3] = m2[2];
    ok = ok && encode_map(st, &m2[4], has_shared ? a.Ws_down : a.W_down, has_shared ? a.I_s : a.I, a.d, 1,
                          sc.pair ? 128 : bn2);
    m2[5] = m2[4];
    // 64-row weight boxes for the half-height tiles of the CTA-pair kernel (phase 1 only)
    if (sc.pair) {
        ok = ok && encode_map(st, &m1[6], a.W_gate, a.d, a.I, a.E, 64);
        ok = ok && encode_map(st, &m1[7], a.W_up, a.d, a.I, a.E, 64);
        ok = ok && encode_map(st, &m1[8], has_shared ? a.Ws_gate : dummy, a.d, has_shared ? a.I_s : a.T, 1, 64);
        ok = ok && encode_map(st, &m1[9], has_shared ? a.Ws_up : dummy, a.d, has_shared ? a.I_s : a.T, 1, 64);
        for (int i = 6; i < 10; ++i) m2[i] = m2[2];
    }
    if (!ok) return MOE_ERR_CUDA;

    // ---- tile lists (already built by the fused front end in direct mode)
    if (!sc.direct && !sc.tiles_built) {
        if (launch_chained(build_tiles_kernel, dim3(1), dim3(1024), 0, s, a.chained && !a.begin_event, sc.tb) != cudaSuccess)
            return MOE_ERR_CUDA;
        ++*launches;
    }
    if (a.begin_event) cudaEventRecord(a.begin_event, s);

    // ---- grids: persistent, never more CTAs than tiles can exist
    const int mblk_routed = rows / kTileRows + (rows < a.E ? rows : a.E);
    const int mblk_shared = has_shared ? ceil_div(a.T, kTileRows) : 0;
    const int max1 = mblk_routed * ceil_div(a.I, bn1 / 2) + mblk_shared * ceil_div(has_shared ? a.I_s : 1, bn1 / 2);
    const int max2 = mblk_routed * ceil_div(a.d, bn2) * ks_r + mblk_shared * ceil_div(a.d, bn2) * ks_s;
    const int ctas_per_sm = decode ? 2 : 1;
    const int grid1 = clampi(max1, 1, sm_count * ctas_per_sm);
    const int grid2 = clampi(max2, 1, sm_count * ctas_per_sm);

    TcParams p1{};
    p1.tiles = ws.tiles1; p1.n_tiles = ws.n_tiles; p1.E = a.E;
    p1.N_routed = a.I; p1.N_shared = a.I_s; p1.out_routed = a.h; p1.out_shared = a.h_s;
    p1.slab_stride_routed = 0; p1.slab_stride_shared = 0; p1.status = ws.status;
    p1.pos = sc.direct ? ws.pos : nullptr; p1.pos_stride = a.T;
    TcParams p2{};
    p2.tiles = ws.tiles2; p2.n_tiles = ws.n_tiles + 1; p2.E = a.E;
    p2.N_routed = a.d; p2.N_shared = a.d; p2.out_routed = a.o; p2.out_shared = a.o_s;
    p2.slab_stride_routed = (unsigned long long)rows * a.d;
    p2.slab_stride_shared = (unsigned long long)a.T * a.d;
    p2.status = ws.status;
    p2.pos = nullptr; p2.pos_stride = 0;
    p2.row_map = a.o_index; p2.row_map_n = rows;

    cudaError_t e1, e2;
    const bool ch = a.chained && !a.mid_event;
#define LEXI_DECODE_PAIR(BN_, AR_, ST_, CTAS_)                                                     \
    do {                                                                                           \
        e1 = launch_tc<1, BN_, AR_, ST_, CTAS_, __nv_bfloat16>(m1, p1, grid1, s, ch);              \
        if (a.mid_event) cudaEventRecord(a.mid_event, s);                                          \
        e2 = launch_tc<2, BN_, AR_, ST_, CTAS_, float>(m2, p2, grid2, s, ch);                      \
    } while (0)
    if (decode) {
        if (a_rows == 32) LEXI_DECODE_PAIR(128, 32, 5, 2);
        else if (a_rows == 64) LEXI_DECODE_PAIR(128, 64, 4, 2);
        else LEXI_DECODE_PAIR(128, 128, 3, 2);
#undef LEXI_DECODE_PAIR
        layout->o_is_f32 = 1;
    } else if (sc.pair) {
        const int rows_t = 2 * kTileRows;
        const int pr = rows / rows_t + (rows < a.E ? rows : a.E), ps = has_shared ? ceil_div(a.T, rows_t) : 0;
        const int pairs1 = pr * ceil_div(a.I, 128) + ps * ceil_div(has_shared ? a.I_s : 1, 128);
        const int pairs2 = (pr + ps) * ceil_div(a.d, 256);
        e1 = launch_tc_pair<1, __nv_bfloat16>(m1, p1, pairs1, s, ch);
        if (a.mid_event) cudaEventRecord(a.mid_event, s);
        e2 = launch_tc_pair<2, float>(m2, p2, pairs2, s, ch);
        layout->o_is_f32 = 1;
    } else {
        e1 = launch_tc<1, 256, 128, 4, 1, __nv_bfloat16>(m1, p1, grid1, s, ch);
        if (a.mid_event) cudaEventRecord(a.mid_event, s);
        // expert outputs stay fp32: with bf16 here the error before the output rounding doubles
        // (1.9e-2 rms on the Qwen-shaped layer, against the 2e-2 bound)
        e2 = launch_tc<2, 256, 128, 4, 1, float>(m2, p2, grid2, s, ch);
        layout->o_is_f32 = 1;
    }
    *launches += 2;
    if (e1 != cudaSuccess || e2 != cudaSuccess) return MOE_ERR_CUDA;
    layout->o_slabs = ks_r;
    layout->o_slab_stride = (size_t)rows * a.d;
    layout->os_slabs = ks_s;
    layout->os_slab_stride = (size_t)a.T * a.d;
    return MOE_OK;
}

}  // namespace lexi
