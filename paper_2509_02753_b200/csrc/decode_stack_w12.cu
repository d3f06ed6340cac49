// The one-launch decode kernel with 12 warps per CTA (168 registers a thread, more bytes in flight).
#define LEXI_FUSED_WARPS 12
#include "decode_stack_body.cuh"
