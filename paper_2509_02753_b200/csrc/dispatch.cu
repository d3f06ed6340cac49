// Dispatch: group the (token, slot) pairs by expert.  The paper (Introduction; Section 3)
// only says that tokens are routed to their top-k experts and that the per-expert token load
// decides the time; the tables built here are the integer definition of that grouping:
//   counts[e], offsets = exclusive scan, perm = pairs in expert-major order with ascending
//   token inside an expert (a stable counting sort), inv_perm = its inverse,
// followed by the gather of the token rows into that order.
//
// Everything is deterministic: ranks come from warp ballots over pairs taken in order, never
// from the arrival order of atomics.
#include <atomic>
#include <cstdlib>

#include "moe_internal.h"
#include "tile_build.cuh"

namespace lexi {

// Each warp owns kPairsPerPart consecutive pairs.  Pass 1: histogram of the part.
__global__ void __launch_bounds__(256) dispatch_count_kernel(DispatchArgs a, int n_pairs, int n_parts) {
    pdl_trigger();
    pdl_wait();
    __shared__ int32_t hist[8][kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int part = blockIdx.x * 8 + warp;
    for (int e = lane; e < a.E; e += 32) hist[warp][e] = 0;
    __syncwarp();
    if (part < n_parts) {
        const int p0 = part * kPairsPerPart;
        const int p1 = min(p0 + kPairsPerPart, n_pairs);
        for (int p = p0 + lane; p < p1; p += 32) {
            const int e = a.topk_idx[p];
            if ((unsigned)e < (unsigned)a.E) atomicAdd(&hist[warp][e], 1);
            else atomicOr(a.status, kStatusBadIndex);
        }
        __syncwarp();
        for (int e = lane; e < a.E; e += 32) a.part_hist[(size_t)part * a.E + e] = hist[warp][e];
    }
}

// Pass 2 (one block): counts, offsets, and for every (part, expert) the first output row.
// Thread (e, seg): expert e = tid % 128, seg = tid / 128 owns one of 8 contiguous ranges of parts,
// so the serial walk over the parts is 8 times shorter and loads are coalesced over e.
constexpr int kScanSegs = 8;
__global__ void __launch_bounds__(kMaxExperts * kScanSegs) dispatch_scan_kernel(DispatchArgs a, int n_parts) {
    pdl_trigger();
    pdl_wait();
    __shared__ int32_t seg_sum[kScanSegs][kMaxExperts];
    __shared__ int32_t off[kMaxExperts + 1];
    const int e = threadIdx.x % kMaxExperts, seg = threadIdx.x / kMaxExperts;
    const int per = (n_parts + kScanSegs - 1) / kScanSegs;
    const int p_begin = min(seg * per, n_parts), p_end = min(p_begin + per, n_parts);
    int total = 0;
    if (e < a.E)
        for (int p = p_begin; p < p_end; ++p) total += a.part_hist[(size_t)p * a.E + e];
    seg_sum[seg][e] = total;
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int i = 0; i < a.E; ++i) {
            off[i] = run;
            for (int sg = 0; sg < kScanSegs; ++sg) run += seg_sum[sg][i];
        }
        off[a.E] = run;
    }
    __syncthreads();
    if (e < a.E) {
        int run = off[e];
        for (int sg = 0; sg < seg; ++sg) run += seg_sum[sg][e];
        if (seg == 0) {
            a.counts[e] = off[e + 1] - off[e];
            a.offsets[e] = off[e];
        }
        for (int p = p_begin; p < p_end; ++p) {
            const int c = a.part_hist[(size_t)p * a.E + e];
            a.part_hist[(size_t)p * a.E + e] = run;
            run += c;
        }
    }
    if (threadIdx.x == 0) a.offsets[a.E] = off[a.E];
}

// Pass 3: each warp walks its part in order, 32 pairs at a time; pairs of the same expert
// inside a step are ranked by lane (ballot), across steps by a per-warp cursor.
__global__ void __launch_bounds__(256) dispatch_scatter_kernel(DispatchArgs a, int n_pairs, int n_parts) {
    pdl_trigger();
    pdl_wait();
    __shared__ int32_t cursor[8][kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int part = blockIdx.x * 8 + warp;
    if (part >= n_parts) return;
    for (int e = lane; e < a.E; e += 32) cursor[warp][e] = a.part_hist[(size_t)part * a.E + e];
    __syncwarp();
    const int p0 = part * kPairsPerPart;
    const int p1 = min(p0 + kPairsPerPart, n_pairs);
    for (int base = p0; base < p1; base += 32) {
        const int p = base + lane;
        const bool valid = p < p1;
        int e = valid ? a.topk_idx[p] : -1;
        if (valid && (unsigned)e >= (unsigned)a.E) e = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        const int leader = __ffs(peers) - 1;
        int first = 0;
        if (e >= 0 && lane == leader) {
            first = cursor[warp][e];
            cursor[warp][e] = first + __popc(peers);
        }
        first = __shfl_sync(0xffffffffu, first, leader);
        if (e >= 0) {
            const int r = first + rank;
            a.perm[r] = p;
            a.inv_perm[p] = r;
        }
        __syncwarp();
    }
}

// Cluster variant: the three passes in ONE launch for calls of any size the layer path sees.  A
// cluster of 8 CTAs shares the pairs (CTA c the c-th eighth, warp w of it a contiguous run), the
// per-CTA totals meet through distributed shared memory, and every CTA then knows where its first
// row of each expert lies: expert-major, inside an expert CTA by CTA, warp by warp, pair by pair -
// the same stable order as the other forms.  Ranks are ballot ranks (no atomics).
// When asked, the eight CTAs also build an eighth each of the tile lists of the tensor-core GEMMs.
constexpr int kDispatchClusterCtas = 8;

__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }

__global__ void __launch_bounds__(1024) dispatch_cluster_kernel(DispatchArgs a, int n_pairs, TileBuildArgs tb, int build) {
    __shared__ int32_t hist[32][kMaxExperts];
    __shared__ int32_t tot_s[kMaxExperts];                       // this CTA's pairs per expert (read by the other CTAs)
    __shared__ int32_t first_s[kMaxExperts];                     // pairs of an expert in the CTAs before this one
    __shared__ int32_t cnt_s[kMaxExperts + 1], off_s[kMaxExperts + 1], part_s[32];
    __shared__ TileBuildSmem tb_sm;
    pdl_trigger();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int n_warps = kDispatchClusterCtas * 32;
    const int per_warp = (((n_pairs + n_warps - 1) / n_warps) + 31) / 32 * 32;
    const int gw = (int)rank * 32 + warp;
    const int p0 = (int)min((long long)gw * per_warp, (long long)n_pairs), p1 = min(p0 + per_warp, n_pairs);
    for (int e = lane; e < kMaxExperts; e += 32) hist[warp][e] = 0;
    __syncwarp();
    pdl_wait();
    // pass 1: histogram of the warp's run; pairs of one expert inside a step are counted by their leader
    for (int base = p0; base < p1; base += 128) {
        int ev[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int p = base + u * 32 + lane;
            ev[u] = p < p1 ? a.topk_idx[p] : -1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            int e = ev[u];
            if (e != -1 && (unsigned)e >= (unsigned)a.E) { atomicOr(a.status, kStatusBadIndex); e = -1; }
            const unsigned peers = __match_any_sync(0xffffffffu, e);
            if (e >= 0 && lane == __ffs(peers) - 1) hist[warp][e] += __popc(peers);
            __syncwarp();
        }
    }
    __syncthreads();
    if (threadIdx.x < kMaxExperts) {
        const int e = threadIdx.x;
        int run = 0;
#pragma unroll 8
        for (int w = 0; w < 32; ++w) {
            const int c = hist[w][e];
            hist[w][e] = run;
            run += c;
        }
        tot_s[e] = run;
    }
    cluster_arrive_release();
    cluster_wait_acquire();
    if (threadIdx.x < kMaxExperts) {
        const int e = threadIdx.x;
        const uint32_t mine = (uint32_t)__cvta_generic_to_shared(&tot_s[e]);
        int total = 0, before = 0;
#pragma unroll
        for (int c = 0; c < kDispatchClusterCtas; ++c) {
            uint32_t remote;
            int v;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(mine), "r"(c));
            asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
            total += v;
            before += c < (int)rank ? v : 0;
        }
        cnt_s[e] = e < a.E ? total : 0;
        first_s[e] = before;
    }
    cluster_arrive_release();      // this CTA has read the others' totals; waited for before it exits
    __syncthreads();
    if (warp == 0) {
        int c[kExpertsPerLane], sum = 0;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane * kExpertsPerLane + j;
            c[j] = e < a.E ? cnt_s[e] : 0;
            sum += c[j];
        }
        // exclusive prefix over the lanes: the sums of the lanes before this one, read from shared
        // memory (32 independent loads instead of a chain of five shuffle rounds)
        part_s[lane] = sum;
        __syncwarp();
        int run = 0, incl = 0;
#pragma unroll 8
        for (int l = 0; l < 32; ++l) {
            const int v = part_s[l];
            run += l < lane ? v : 0;
            incl += l <= lane ? v : 0;
        }
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane * kExpertsPerLane + j;
            if (e < a.E) {
                off_s[e] = run;
                if (rank == 0) { a.counts[e] = c[j]; a.offsets[e] = run; }
            }
            run += c[j];
        }
        if (lane == 31) {
            off_s[a.E] = incl;
            if (rank == 0) a.offsets[a.E] = incl;
        }
    }
    __syncthreads();
    // pass 2: ranked placement; off_s[e] + first_s[e] + hist[warp][e] is the warp's cursor for expert e
    for (int base = p0; base < p1; base += 128) {
        int ev[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int p = base + u * 32 + lane;
            ev[u] = p < p1 ? a.topk_idx[p] : -1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int p = base + u * 32 + lane;
            int e = ev[u];
            if ((unsigned)e >= (unsigned)a.E) e = -1;
            const unsigned peers = __match_any_sync(0xffffffffu, e);
            const int leader = __ffs(peers) - 1;
            int first = 0;
            if (e >= 0 && lane == leader) {
                first = hist[warp][e];
                hist[warp][e] = first + __popc(peers);
                first += off_s[e] + first_s[e];
            }
            first = __shfl_sync(0xffffffffu, first, leader);
            if (e >= 0) {
                const int r = first + __popc(peers & ((1u << lane) - 1u));
                a.perm[r] = p;
                a.inv_perm[p] = r;
            }
            __syncwarp();
        }
    }
    if (build) {
        __syncthreads();
        build_tiles_block(tb, cnt_s, off_s, tb_sm, (int)rank, kDispatchClusterCtas);
    }
    cluster_wait_acquire();
}

// The tile lists alone, from tables that are already in global memory (one block).
__global__ void __launch_bounds__(1024) tile_lists_kernel(TileBuildArgs tb) {
    __shared__ int32_t cnt_s[kMaxExperts + 1], off_s[kMaxExperts + 1];
    __shared__ TileBuildSmem tb_sm;
    pdl_trigger();
    pdl_wait();
    for (int e = threadIdx.x; e <= tb.E; e += blockDim.x) {
        cnt_s[e] = e < tb.E ? tb.counts[e] : 0;
        off_s[e] = tb.offsets[e];
    }
    __syncthreads();
    build_tiles_block(tb, cnt_s, off_s, tb_sm);
}

cudaError_t launch_dispatch(const DispatchArgs &a, cudaStream_t s, uint64_t *launches, bool chained);

// A device (or a share of one) that cannot run 8 CTAs of 1024 threads as one cluster gets the
// three-kernel form followed by a one-block tile builder; LEXI_DISPATCH_CLUSTER=0 asks for that too.
cudaError_t launch_dispatch_cluster(const DispatchArgs &a, cudaStream_t s, uint64_t *launches, bool chained,
                                    const TileBuildArgs *tiles) {
    const int n_pairs = a.T * a.k;
    if (n_pairs <= 0) return cudaSuccess;
    static const bool env_off = [] { const char *v = getenv("LEXI_DISPATCH_CLUSTER"); return v && v[0] == '0'; }();
    static std::atomic<int> usable[64];            // per device: 0 unknown, 1 yes, -1 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); dev = -1; }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(kDispatchClusterCtas); cfg.blockDim = dim3(1024); cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kDispatchClusterCtas; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    int state = env_off || dev < 0 ? -1 : usable[dev].load(std::memory_order_acquire);
    if (state == 0) {
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, dispatch_cluster_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
        state = n >= 1 ? 1 : -1;
        usable[dev].store(state, std::memory_order_release);
    }
    if (state == 1) {
        cfg.numAttrs = chained ? 2 : 1;
        const cudaError_t e = cudaLaunchKernelEx(&cfg, dispatch_cluster_kernel, a, n_pairs,
                                                 tiles ? *tiles : TileBuildArgs{}, tiles ? 1 : 0);
        ++*launches;
        return e;
    }
    cudaError_t e = launch_dispatch(a, s, launches, chained);
    if (e == cudaSuccess && tiles) {
        e = launch_chained(tile_lists_kernel, dim3(1), dim3(1024), 0, s, chained, *tiles);
        ++*launches;
    }
    return e;
}

cudaError_t launch_dispatch(const DispatchArgs &a, cudaStream_t s, uint64_t *launches, bool chained) {
    const int n_pairs = a.T * a.k;
    if (n_pairs <= 0) return cudaSuccess;
    const int n_parts = (n_pairs + kPairsPerPart - 1) / kPairsPerPart;
    const int grid = (n_parts + 7) / 8;
    cudaError_t e = launch_chained(dispatch_count_kernel, dim3(grid), dim3(256), 0, s, chained, a, n_pairs, n_parts);
    if (e == cudaSuccess)
        e = launch_chained(dispatch_scan_kernel, dim3(1), dim3(kMaxExperts * kScanSegs), 0, s, chained, a, n_parts);
    if (e == cudaSuccess)
        e = launch_chained(dispatch_scatter_kernel, dim3(grid), dim3(256), 0, s, chained, a, n_pairs, n_parts);
    *launches += 3;
    return e;
}

// Gather: x_perm[r, :] = x[perm[r] / k, :], one warp per row, 16-byte loads and stores.
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4 *__restrict__ x,
                                                          const int32_t *__restrict__ perm,
                                                          int n_rows, int k, int vec_per_row,
                                                          uint4 *__restrict__ x_perm) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int warps = gridDim.x * 8;
    for (int r = blockIdx.x * 8 + (threadIdx.x >> 5); r < n_rows; r += warps) {
        const int t = perm[r] / k;
        const uint4 *src = x + (size_t)t * vec_per_row;
        uint4 *dst = x_perm + (size_t)r * vec_per_row;
        for (int v = lane; v < vec_per_row; v += 32) dst[v] = src[v];
    }
}

cudaError_t launch_gather(const void *x, const int32_t *perm, int n_rows, int k, int d, int dtype,
                          void *x_perm, cudaStream_t s, uint64_t *launches, bool chained) {
    if (n_rows <= 0) return cudaSuccess;
    const int bytes_per_row = d * (dtype == MOE_BF16 ? 2 : 4);
    const int grid = min((n_rows + 7) / 8, 148 * 8);
    const cudaError_t e = launch_chained(gather_rows_kernel, dim3(grid), dim3(256), 0, s, chained,
                                         (const uint4 *)x, perm, n_rows, k, bytes_per_row / 16, (uint4 *)x_perm);
    ++*launches;
    return e;
}

// Expert parallelism, sending side, as plain stores into the owners' memory: the rows of this
// rank's (token, slot) pairs, taken in expert order (perm), are written straight to the place they
// have in the OWNER's expert-major buffer - local experts ascending, inside an expert the source
// ranks ascending, inside a source the pairs in their stable order - so that the owner can run its
// grouped GEMMs on what arrived, with no exchange call and no regrouping copy.  all_counts
// [world, E]: pairs per (source rank, global expert), the same on every rank.  peers: one base pointer
// per rank (its arrival buffer: this GPU's own memory for `rank`, peer-mapped memory for the others).
// Every block redoes the small prefix sums in shared memory.
constexpr int kMaxRegroupBlocks = 1024;      // (local expert, source rank) blocks an expert-parallel rank may have
struct PeerRows { void *base[kMaxPeers]; int32_t capacity[kMaxPeers]; };   // arrival buffers and their sizes in rows

__global__ void __launch_bounds__(256) send_rows_kernel(const uint4 *__restrict__ x, const int32_t *__restrict__ perm,
                                                        int n_rows, int k, int vec_per_row,
                                                        const int32_t *__restrict__ all_counts, int E, int rank, int world,
                                                        PeerRows peers, int32_t *status) {
    __shared__ int32_t my_off[kMaxExperts + 1];       // this rank's pairs: first packed row of each expert
    __shared__ int32_t dest_start[kMaxExperts];       // row in the owner's buffer where this rank's rows of expert e begin
    const int e_loc = E / world;
    if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) { my_off[e] = run; run += max(all_counts[rank * E + e], 0); }
        my_off[E] = run;
    }
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        const int first = e / e_loc * e_loc;          // the owner's first expert
        int start = 0;
        for (int e2 = first; e2 < e; ++e2)
            for (int sr = 0; sr < world; ++sr) start += max(all_counts[sr * E + e2], 0);
        for (int sr = 0; sr < rank; ++sr) start += max(all_counts[sr * E + e], 0);
        dest_start[e] = start;
    }
    __syncthreads();
    if (my_off[E] != n_rows) {                        // the counts do not describe the rows given: nothing is sent
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, kStatusBadIndex);
        return;
    }
    const int lane = threadIdx.x & 31;
    const int warps = gridDim.x * 8;
    for (int r = blockIdx.x * 8 + (threadIdx.x >> 5); r < n_rows; r += warps) {
        int lo = 0, hi = E - 1;                       // last expert whose first row is <= r
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (my_off[mid] <= r) lo = mid; else hi = mid - 1;
        }
        const int e = lo;
        const int dst_row = dest_start[e] + (r - my_off[e]);
        if (dst_row >= peers.capacity[e / e_loc]) {   // the owner's buffer is too small: flagged, row dropped
            if (lane == 0) atomicOr(status, kStatusBadIndex);
            continue;
        }
        const uint4 *src = x + (size_t)(perm[r] / k) * vec_per_row;
        uint4 *dst = reinterpret_cast<uint4 *>(peers.base[e / e_loc]) + (size_t)dst_row * vec_per_row;
        for (int v = lane; v < vec_per_row; v += 32) dst[v] = src[v];
    }
}

cudaError_t launch_send_rows(const void *x, const int32_t *perm, int n_rows, int k, int d, int dtype,
                             const int32_t *all_counts, int E, int rank, int world, void *const *peer_rows,
                             const int32_t *capacity_rows, int32_t *status, cudaStream_t s, uint64_t *launches) {
    PeerRows peers{};
    for (int r = 0; r < world; ++r) { peers.base[r] = peer_rows[r]; peers.capacity[r] = capacity_rows[r]; }
    const int bytes_per_row = d * (dtype == MOE_BF16 ? 2 : 4);
    const int grid = n_rows > 0 ? min((n_rows + 7) / 8, 148 * 8) : 1;
    send_rows_kernel<<<grid, 256, 0, s>>>((const uint4 *)x, perm, n_rows, k, bytes_per_row / 16, all_counts, E, rank, world,
                                          peers, status);
    ++*launches;
    return cudaGetLastError();
}

// Expert parallelism, the way back, as plain stores: the owner's fp32 outputs, in the expert-major
// order of its arrival buffer, go straight to the row each pair has in its SOURCE rank's packed
// (expert) order, which is the order that rank's moe_combine indexes with inv_perm.  Block (local
// expert e, source s) of the owner's rows starts at blk_start[e * world + s] and belongs at row
// src_off = sum of all_counts[s][0 .. global e) of source s's buffer.
__global__ void __launch_bounds__(256) return_rows_kernel(const uint4 *__restrict__ o_rows, int n_rows, int vec_per_row,
                                                          const int32_t *__restrict__ all_counts, int E, int rank, int world,
                                                          PeerRows peers, int32_t *status) {
    __shared__ int32_t blk_start[kMaxRegroupBlocks + 1], src_off[kMaxRegroupBlocks];
    const int e_loc = E / world, nb = e_loc * world;
    for (int b = threadIdx.x; b < nb; b += blockDim.x) {      // b = local expert * world + source
        const int el = b / world, sr = b - el * world, e = rank * e_loc + el;
        int off = 0;
        for (int e2 = 0; e2 < e; ++e2) off += max(all_counts[sr * E + e2], 0);
        src_off[b] = off;
    }
    if (threadIdx.x == 0) {
        int run = 0;
        for (int b = 0; b < nb; ++b) {
            const int el = b / world, sr = b - el * world;
            blk_start[b] = run;
            run += max(all_counts[sr * E + rank * e_loc + el], 0);
        }
        blk_start[nb] = run;
    }
    __syncthreads();
    if (blk_start[nb] != n_rows) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, kStatusBadIndex);
        return;
    }
    const int lane = threadIdx.x & 31;
    const int warps = gridDim.x * 8;
    for (int r = blockIdx.x * 8 + (threadIdx.x >> 5); r < n_rows; r += warps) {
        int lo = 0, hi = nb - 1;                              // last block that starts at or before r
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (blk_start[mid] <= r) lo = mid; else hi = mid - 1;
        }
        const int sr = lo % world;
        const int dst_row = src_off[lo] + (r - blk_start[lo]);
        if (dst_row >= peers.capacity[sr]) {
            if (lane == 0) atomicOr(status, kStatusBadIndex);
            continue;
        }
        const uint4 *src = o_rows + (size_t)r * vec_per_row;
        uint4 *dst = reinterpret_cast<uint4 *>(peers.base[sr]) + (size_t)dst_row * vec_per_row;
        for (int v = lane; v < vec_per_row; v += 32) dst[v] = src[v];
    }
}

cudaError_t launch_return_rows(const float *o_rows, int n_rows, int d, const int32_t *all_counts, int E, int rank, int world,
                               void *const *peer_rows, const int32_t *capacity_rows, int32_t *status, cudaStream_t s,
                               uint64_t *launches) {
    PeerRows peers{};
    for (int r = 0; r < world; ++r) { peers.base[r] = peer_rows[r]; peers.capacity[r] = capacity_rows[r]; }
    const int grid = n_rows > 0 ? min((n_rows + 7) / 8, 148 * 8) : 1;
    return_rows_kernel<<<grid, 256, 0, s>>>((const uint4 *)o_rows, n_rows, d * 4 / 16, all_counts, E, rank, world, peers, status);
    ++*launches;
    return cudaGetLastError();
}

// Expert parallelism, receiving side: rows arrive source-major (all rows of source rank 0, then
// rank 1, ...; inside a source the local experts ascend) and the grouped GEMMs want them
// expert-major (inside an expert the sources in rank order).  recv_counts [world, E] = rows per
// (source, local expert).  to_em[p] = arrival index of the row at expert-major position p, inv its
// inverse, per_expert[e] = rows of local expert e.  Every CTA redoes the two small scans over the
// world x E blocks in shared memory and then copies index ranges of its share of the blocks.
__global__ void __launch_bounds__(256) regroup_index_kernel(const int32_t *__restrict__ recv_counts, int world, int E,
                                                            int n_rows, int32_t *to_em, int32_t *inv,
                                                            int32_t *per_expert, int32_t *status) {
    __shared__ int32_t len[kMaxRegroupBlocks], arr_start[kMaxRegroupBlocks], out_start[kMaxRegroupBlocks];
    __shared__ int32_t total;
    const int nb = world * E;
    for (int b = threadIdx.x; b < nb; b += blockDim.x) len[b] = max(recv_counts[b], 0);      // b = source * E + expert
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int b = 0; b < nb; ++b) { arr_start[b] = run; run += len[b]; }                 // arrival order
        total = run;
        run = 0;
        for (int e = 0; e < E; ++e)
            for (int sr = 0; sr < world; ++sr) { out_start[sr * E + e] = run; run += len[sr * E + e]; }   // expert-major order
    }
    __syncthreads();
    const bool bad = total != n_rows;
    if (blockIdx.x == 0) {
        if (bad && threadIdx.x == 0) atomicOr(status, kStatusBadIndex);
        for (int e = threadIdx.x; e < E; e += blockDim.x) {
            int c = 0;
            for (int sr = 0; sr < world; ++sr) c += len[sr * E + e];
            per_expert[e] = bad ? 0 : c;
        }
    }
    if (bad) return;
    for (int b = blockIdx.x; b < nb; b += gridDim.x) {
        const int a0 = arr_start[b], o0 = out_start[b];
        for (int i = threadIdx.x; i < len[b]; i += blockDim.x) {
            to_em[o0 + i] = a0 + i;
            inv[a0 + i] = o0 + i;
        }
    }
}

cudaError_t launch_regroup_index(const int32_t *recv_counts, int world, int E, int n_rows, int32_t *to_em, int32_t *inv,
                                 int32_t *per_expert, int32_t *status, cudaStream_t s, uint64_t *launches) {
    const int nb = world * E;
    regroup_index_kernel<<<nb < 296 ? nb : 296, 256, 0, s>>>(recv_counts, world, E, n_rows, to_em, inv, per_expert, status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lexi

// ---------------------------------------------------------------------------------------
// Dispatch tables without any allocation.
//
// Some callers of this library may not allocate device memory at the point where they need
// the dispatch tables: a serving loop that must not hit the implicit device synchronisation of
// cudaMalloc/cudaFree between decoding steps, or a host component that was handed a stream and
// buffers by its framework but has no allocator of its own and so cannot create a plan (a plan
// owns a cudaMalloc'ed workspace).  For them the scratch of the three dispatch passes (the
// per-partition histograms, the inverse permutation and a status word) lives in the fixed
// array below, which every GPU that loads this library carries until the process exits.
// ---------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxPairs = 65536;                                   // T * k_l limit
constexpr int kStaticMaxParts = kStaticMaxPairs / lexi::kPairsPerPart;   // 256
constexpr int kStaticStatusInts = 64;                                    // status word, padded to 256 B
constexpr int kStaticHistInts = kStaticMaxParts * lexi::kMaxExperts;     // 32768
constexpr int kStaticScratchInts = kStaticStatusInts + kStaticHistInts + kStaticMaxPairs;   // 393,472 bytes

static __device__ __align__(256) int32_t g_dispatch_scratch[kStaticScratchInts];

// The array's name is only a host-side handle; the device address has to be asked for, once per
// device, with that device current.
constexpr int kMaxDevices = 64;
std::atomic<int32_t *> g_scratch_addr[kMaxDevices];

int32_t *static_scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return nullptr; }
    int32_t *ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        // two host threads may both get here on their first call; both are told the same address
        if (cudaGetSymbolAddress((void **)&ptr, g_dispatch_scratch) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}

}  // namespace

extern "C" int moe_dispatch_tables_static(const int32_t *topk_idx, int32_t T, int32_t k_l, int32_t E,
                                          int32_t *counts, int32_t *offsets, int32_t *perm,
                                          void *cuda_stream) {
    if (!topk_idx || !counts || !offsets || !perm) return MOE_ERR_INVALID_ARG;
    if (T < 0 || k_l < 1 || E < 1 || k_l > E) return MOE_ERR_INVALID_ARG;
    if (E > lexi::kMaxExperts || (int64_t)T * k_l > kStaticMaxPairs) return MOE_ERR_SHAPE;
    int32_t *scratch = static_scratch_for_current_device();
    if (!scratch) return MOE_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the array keeps whatever the previous call left; only the status word has to start at zero
    // (histograms and the inverse permutation are fully rewritten for the sizes of this call)
    if (cudaMemsetAsync(scratch, 0, sizeof(int32_t), s) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    lexi::DispatchArgs a{topk_idx, T, k_l, E, counts, offsets, perm,
                         scratch + kStaticStatusInts + kStaticHistInts,   // inverse permutation
                         scratch + kStaticStatusInts,                     // per-partition histograms
                         scratch};                                        // status word
    if (T == 0) {
        if (cudaMemsetAsync(counts, 0, sizeof(int32_t) * E, s) != cudaSuccess ||
            cudaMemsetAsync(offsets, 0, sizeof(int32_t) * (E + 1), s) != cudaSuccess) {
            cudaGetLastError();
            return MOE_ERR_CUDA;
        }
        return MOE_OK;
    }
    uint64_t launches = 0;
    return lexi::launch_dispatch(a, s, &launches, false) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
