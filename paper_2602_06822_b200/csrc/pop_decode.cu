// Fused persistent decode kernel (placeholder until the kernel lands: defers to the plain path).
#include "pop_common.cuh"

int pop_launch_decode(pop_partition* p, const void* x, int B, int k, void* y, uint8_t* mask_out,
                      int32_t* sel_out, cudaStream_t st) {
    (void)p; (void)x; (void)B; (void)k; (void)y; (void)mask_out; (void)sel_out; (void)st;
    return POP_ERR_UNSUPPORTED;
}
