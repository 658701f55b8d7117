// Device helpers shared by the register-dequant kernels: the m16n8k16 BF16 MMA, the nibble-to-BF16
// conversion of the packed layout (Eq. 3 codes, offset-binary), block sums of activations, and the
// programmatic-dependent-launch controls.
#pragma once
#include <stdint.h>
#include <cuda_runtime.h>

namespace exmoe {

__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two offset-binary nibbles (bits s..s+3 of each 16-bit half) -> bf16x2 of 128 + u = 136 + q:
// 0x4300 | u is that BF16 value exactly (one shift and one lop3 per pair of codes).
__device__ __forceinline__ uint32_t code_pair(uint32_t w, int s) {
    uint32_t r;
    asm("lop3.b32 %0, %1, 0x000f000f, 0x43004300, 0xea;" : "=r"(r) : "r"(w >> s));   // (a & b) | c
    return r;
}
// sum of the 8 BF16 values of a 16-byte chunk, in binary32
__device__ __forceinline__ float sum8_bf16(const uint4& v) {
    const uint32_t r[4] = {v.x, v.y, v.z, v.w};
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) s += __uint_as_float(r[i] << 16) + __uint_as_float(r[i] & 0xffff0000u);
    return s;
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace exmoe
