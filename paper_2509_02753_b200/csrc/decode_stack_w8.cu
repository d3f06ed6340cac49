// The one-launch decode kernel with 8 warps per CTA (255 registers a thread, no spills).
#define LEXI_FUSED_WARPS 8
#include "decode_stack_body.cuh"
