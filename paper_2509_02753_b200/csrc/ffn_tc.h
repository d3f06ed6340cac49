// Tensor-core (tcgen05 / TMEM / TMA) schedules of the expert FFNs: host-side interface.
#pragma once

#include "moe_internal.h"
#include "tile_build.cuh"

namespace lexi {

struct TcState {
    void *encode_fn = nullptr;   // cuTensorMapEncodeTiled, resolved through the runtime
    int max_smem_optin = 0;
    bool ready = false;
};

// How the combine step has to read the expert outputs a schedule produced.
struct TcOutputLayout {
    int o_is_f32 = 1;
    int o_slabs = 1;
    size_t o_slab_stride = 0;
    int os_slabs = 1;
    size_t os_slab_stride = 0;
};

bool   tc_shape_ok(const moe_config_t &c);
int    tc_max_slabs(const moe_config_t &c);          // most split-K slabs of the routed output
int    tc_max_shared_slabs(const moe_config_t &c);   // ... of the shared-expert output
size_t tc_o_elems(const moe_config_t &c, int slabs);     // fp32-sized elements to hold `o`
size_t tc_os_elems(const moe_config_t &c, int slabs);    // ... `o_s`
size_t tc_max_tiles(const moe_config_t &c, int phase);   // capacity of a tile list
int    tc_state_init(TcState *st, const moe_config_t &c);
cudaError_t launch_wait_probe(int32_t *status, unsigned long long limit_ns, cudaStream_t s);
// Encodes a TMA tensor map (into the 128-byte CUtensorMap at `map`) of a bf16 tensor
// [groups, rows, K] with K contiguous: box 64 x box_rows x 1, 128-byte swizzle, zero fill outside.
bool   tc_encode_bf16_map(const TcState *st, void *map, const void *ptr, uint64_t K, uint64_t rows,
                          uint64_t groups, uint32_t box_rows);
// Tensor-core router for large T (router_tc.cu); returns false if the shape is not covered.
bool   tc_router_supported(const TcState *st, const RouterArgs &a);
cudaError_t launch_router_tc(const TcState *st, const RouterArgs &a, int sm_count, cudaStream_t s,
                             uint64_t *launches);
// Tile shapes, split-K factors and the tile-list recipe of one call.
struct TcSchedule {
    bool decode = false, direct = false;
    bool pair = false;           // prefill GEMMs on CTA pairs (256-row tiles)
    bool tiles_built = false;    // the tile lists were already built by the dispatch or front-end kernel
    int bn1 = 256, bn2 = 256, a_rows = 128, ks_r = 1, ks_s = 1, kchunk_r = 64, kchunk_s = 64;
    TileBuildArgs tb{};
};
void   tc_make_schedule(const moe_config_t &c, const Workspace &ws, const FfnArgs &a, int schedule,
                        bool direct, int sm_count, TcSchedule *out);
int    tc_ffn_forward(TcState *st, const moe_config_t &c, const Workspace &ws, const FfnArgs &a,
                      const TcSchedule &sc, int sm_count, cudaStream_t s, uint64_t *launches,
                      TcOutputLayout *layout);

// Fused front end of small decode calls (decode_front.cu): router, top-k, dispatch tables, position
// table and both tile lists in one launch; the last block to finish the logits does the rest.
struct FrontArgs {
    RouterArgs r;
    int32_t *counts, *offsets, *perm, *inv_perm, *pos, *ticket;
    TileBuildArgs tb;
};
constexpr int kFrontMaxTokens = 128;
constexpr int kFrontMaxPairs = 2048;
cudaError_t launch_decode_front(const FrontArgs &a, cudaStream_t s, uint64_t *launches);

}  // namespace lexi
