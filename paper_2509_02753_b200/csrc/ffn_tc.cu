#include "ffn_tc.h"
namespace lexi {
bool tc_shape_ok(const moe_config_t &) { return false; }
int tc_max_slabs(const moe_config_t &) { return 1; }
int tc_max_shared_slabs(const moe_config_t &) { return 1; }
size_t tc_o_elems(const moe_config_t &c, int slabs) { return (size_t)slabs * c.max_T * c.max_k * c.d; }
size_t tc_os_elems(const moe_config_t &c, int slabs) { return (size_t)slabs * c.max_T * c.d; }
size_t tc_max_tiles(const moe_config_t &, int) { return 1; }
int tc_state_init(TcState *, const moe_config_t &) { return MOE_OK; }
int tc_ffn_forward(TcState *, const moe_config_t &, const Workspace &, const FfnArgs &, int, int, cudaStream_t, uint64_t *, TcOutputLayout *) { return MOE_ERR_NOT_IMPLEMENTED; }
}
