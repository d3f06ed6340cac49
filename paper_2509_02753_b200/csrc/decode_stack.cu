// Host side of the one-launch decode kernel (decode_stack_body.cuh): which of its two builds runs a call.
#include <cstdlib>

#include "moe_internal.h"

namespace lexi {

size_t fused_smem_bytes_w8(int d);
size_t fused_smem_bytes_w12(int d);
cudaError_t fused_prepare_w8(int d);
cudaError_t fused_prepare_w12(int d);
cudaError_t launch_decode_stack_w8(const StackArgs &a, int sm_count, cudaStream_t s, uint64_t *launches);
cudaError_t launch_decode_stack_w12(const StackArgs &a, int sm_count, cudaStream_t s, uint64_t *launches);

size_t fused_smem_bytes(int d) {
    const size_t a = fused_smem_bytes_w8(d), b = fused_smem_bytes_w12(d);
    return a > b ? a : b;
}

cudaError_t fused_prepare(int d) {
    const cudaError_t e = fused_prepare_w8(d);
    return e != cudaSuccess ? e : fused_prepare_w12(d);
}

// 12 warps for shapes whose single experts are so large that a CTA's share of ONE expert exceeds a
// megabyte (the Mixtral shape: 352 MB per expert; measured 3 % faster there at 1 and 8 tokens), 8 warps
// otherwise (measured 3-8 % faster on the Qwen1.5-, OLMoE-, DeepSeek-V2-Lite- and VL2-Tiny-shaped
// stacks at 1 token, equal or better at 8).  LEXI_DECODE_WARPS=8|12 forces one build.
constexpr double kWideExpertBytesPerCta = 1.0e6;

cudaError_t launch_decode_stack(const StackArgs &a, int sm_count, cudaStream_t s, uint64_t *launches) {
    static const char *env = getenv("LEXI_DECODE_WARPS");
    bool wide = 2.0 * 3.0 * a.d * (double)a.I / sm_count > kWideExpertBytesPerCta;
    if (env && env[0] == '8') wide = false;
    if (env && env[0] == '1') wide = true;
    return wide ? launch_decode_stack_w12(a, sm_count, s, launches) : launch_decode_stack_w8(a, sm_count, s, launches);
}

}  // namespace lexi
