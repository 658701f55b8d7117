// Device code shared by the one-launch tiny-batch kernels: streaming loads, the per-block multiply-accumulate chains
// over packed weights (in shared memory or in registers) against ONE activation row, and the block sums of an
// activation row.  The chain of fused multiply-adds over a K range's blocks, in ascending order from zero, and the
// way the block corrections are formed are those of the decode kernels in decode.cu: same bits.
#pragma once
#include "common.cuh"
#include "frag.cuh"
#include "mbar.cuh"

namespace exmoe {

// 16-byte asynchronous copy global -> shared through the load/store path (no register staging, L1 bypassed)
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ uint4 ldg_stream128(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ldg_stream32(const void* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 ldg_early128(const void* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// One K range of NM matrices (gate and up, or down) against ONE activation row: `nb` consecutive 128-wide blocks
// starting at block kb0, weights in shared memory in packed (= fragment) order.  tot[m][0/1] = rows q / q+8 of the
// panel, valid on the lanes with c == 0.  The chain of fused multiply-adds over the range's blocks, in ascending
// order from zero, is the rounding order of the other decode kernels.
template <int NM>
__device__ __forceinline__ void range_chain(const unsigned char* const (&w)[NM], int nb, int kb0,
                                            const unsigned char* xrow, const float* adj, int lane, float (&tot)[NM][2]) {
    const int q = lane >> 2, c = lane & 3;
#pragma unroll
    for (int m = 0; m < NM; ++m) tot[m][0] = tot[m][1] = 0.f;
#pragma unroll 2
    for (int b = 0; b < nb; ++b) {
        float acc[NM][4];
        uint4 wl[NM], wh[NM];
        uint32_t sv[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m) {
            const unsigned char* blk = w[m] + (size_t)b * kBlockBytes;
            wl[m] = *reinterpret_cast<const uint4*>(blk + lane * 16);
            wh[m] = *reinterpret_cast<const uint4*>(blk + 512 + lane * 16);
            sv[m] = *reinterpret_cast<const uint32_t*>(blk + kCodeBytes + q * 4);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[m][i] = 0.f;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int set = 0; set < 2; ++set) {
                const int k0 = (kb0 + b) * kGroup + 64 * h + 32 * set + 8 * c;
                uint4 xb = make_uint4(0, 0, 0, 0);
                if (q == 0) xb = *reinterpret_cast<const uint4*>(xrow + k0 * 2);
#pragma unroll
                for (int m = 0; m < NM; ++m) {
                    const uint4& wv = h ? wh[m] : wl[m];
                    const uint32_t wq = set ? wv.z : wv.x;
                    const uint32_t wq8 = set ? wv.w : wv.y;
                    mma_m16n8k16(acc[m], code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                    mma_m16n8k16(acc[m], code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
                }
            }
        const float cr = adj[kb0 + b];
#pragma unroll
        for (int m = 0; m < NM; ++m) {
            const __half2 sc = *reinterpret_cast<const __half2*>(&sv[m]);
            tot[m][0] = fmaf(__low2float(sc), acc[m][0] + cr, tot[m][0]);
            tot[m][1] = fmaf(__high2float(sc), acc[m][2] + cr, tot[m][1]);
        }
    }
}

// NU units of NB blocks each against ONE activation row, everything unrolled: all weight words are read first, then the
// NU x NB accumulator chains run interleaved (a chain of eight dependent MMAs per block is latency-bound on its own);
// the per-unit sums over the blocks are then formed in ascending order, as everywhere.
template <int NU, int NB>
__device__ __forceinline__ void unit_chains(const unsigned char* const (&w)[NU], const unsigned char* xrow, const float* adj,
                                            int lane, float (&tot)[NU][2]) {
    const int q = lane >> 2, c = lane & 3;
    uint4 wl[NU][NB], wh[NU][NB];
    uint32_t sv[NU][NB];
    float acc[NU][NB][4];
#pragma unroll
    for (int u = 0; u < NU; ++u)
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const unsigned char* blk = w[u] + (size_t)b * kBlockBytes;
            wl[u][b] = *reinterpret_cast<const uint4*>(blk + lane * 16);
            wh[u][b] = *reinterpret_cast<const uint4*>(blk + 512 + lane * 16);
            sv[u][b] = *reinterpret_cast<const uint32_t*>(blk + kCodeBytes + q * 4);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[u][b][i] = 0.f;
        }
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int set = 0; set < 2; ++set)
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const int k0 = b * kGroup + 64 * h + 32 * set + 8 * c;
                uint4 xb = make_uint4(0, 0, 0, 0);
                if (q == 0) xb = *reinterpret_cast<const uint4*>(xrow + k0 * 2);
#pragma unroll
                for (int u = 0; u < NU; ++u) {
                    const uint4& wv = h ? wh[u][b] : wl[u][b];
                    const uint32_t wq = set ? wv.z : wv.x;
                    const uint32_t wq8 = set ? wv.w : wv.y;
                    mma_m16n8k16(acc[u][b], code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                    mma_m16n8k16(acc[u][b], code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
                }
            }
#pragma unroll
    for (int u = 0; u < NU; ++u) {
        tot[u][0] = tot[u][1] = 0.f;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const float cr = adj[b];
            const __half2 sc = *reinterpret_cast<const __half2*>(&sv[u][b]);
            tot[u][0] = fmaf(__low2float(sc), acc[u][b][0] + cr, tot[u][0]);
            tot[u][1] = fmaf(__high2float(sc), acc[u][b][2] + cr, tot[u][1]);
        }
    }
}

// The same chains for NM units that each have their OWN activation row and corrections (units of different token-expert
// pairs): `nb` blocks per unit, x[m] and adj[m] already offset to the unit's K range.  Independent accumulator chains,
// interleaved.
template <int NM>
__device__ __forceinline__ void range_chain_rows(const unsigned char* const (&w)[NM], int nb, const unsigned char* const (&x)[NM],
                                                 const float* const (&adj)[NM], int lane, float (&tot)[NM][2]) {
    const int q = lane >> 2, c = lane & 3;
#pragma unroll
    for (int m = 0; m < NM; ++m) tot[m][0] = tot[m][1] = 0.f;
#pragma unroll 2
    for (int b = 0; b < nb; ++b) {
        float acc[NM][4];
        uint4 wl[NM], wh[NM];
        uint32_t sv[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m) {
            const unsigned char* blk = w[m] + (size_t)b * kBlockBytes;
            wl[m] = *reinterpret_cast<const uint4*>(blk + lane * 16);
            wh[m] = *reinterpret_cast<const uint4*>(blk + 512 + lane * 16);
            sv[m] = *reinterpret_cast<const uint32_t*>(blk + kCodeBytes + q * 4);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[m][i] = 0.f;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int set = 0; set < 2; ++set) {
                const int k0 = b * kGroup + 64 * h + 32 * set + 8 * c;
#pragma unroll
                for (int m = 0; m < NM; ++m) {
                    uint4 xb = make_uint4(0, 0, 0, 0);
                    if (q == 0) xb = *reinterpret_cast<const uint4*>(x[m] + k0 * 2);
                    const uint4& wv = h ? wh[m] : wl[m];
                    const uint32_t wq = set ? wv.z : wv.x;
                    const uint32_t wq8 = set ? wv.w : wv.y;
                    mma_m16n8k16(acc[m], code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                    mma_m16n8k16(acc[m], code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
                }
            }
#pragma unroll
        for (int m = 0; m < NM; ++m) {
            const float cr = adj[m][b];
            const __half2 sc = *reinterpret_cast<const __half2*>(&sv[m]);
            tot[m][0] = fmaf(__low2float(sc), acc[m][0] + cr, tot[m][0]);
            tot[m][1] = fmaf(__high2float(sc), acc[m][2] + cr, tot[m][1]);
        }
    }
}

// adj[kb] = -136 * (sum of the row's block kb), formed chunk by chunk (8 values, then a 16-lane butterfly) exactly
// as the staging loops of the other decode kernels do.  The row is already in shared memory.
__device__ __forceinline__ void block_sums(const unsigned char* row, int n_chunks, float* adj, int warp, int lane, int n_threads) {
    for (int base = warp * 32; base < n_chunks; base += n_threads) {
        const int ck = base + lane;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (ck < n_chunks) v = *reinterpret_cast<const uint4*>(row + ck * 16);
        float sx = sum8_bf16(v);
#pragma unroll
        for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
        if (ck < n_chunks && (ck & 15) == 0) adj[ck >> 4] = -136.f * sx;
    }
}

// One block of the same chain with the gate and up blocks held in REGISTERS: block `b` of the warp's K range (`xr`
// holds just that range of the activation row, adj the block's correction).  Called block by block, in ascending
// order, so that the loads of later blocks can be issued in between.
__device__ __forceinline__ void chain_block_regs(const uint4 (&wb)[2][2], const uint32_t (&sb)[2], float adj, int b,
                                                 const unsigned char* xr, int lane, float (&tot)[2][2]) {
    const int q = lane >> 2, c = lane & 3;
    float acc[2][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[m][i] = 0.f;
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int set = 0; set < 2; ++set) {
            const int k0 = b * kGroup + 64 * h + 32 * set + 8 * c;
            uint4 xb = make_uint4(0, 0, 0, 0);
            if (q == 0) xb = *reinterpret_cast<const uint4*>(xr + k0 * 2);
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                const uint32_t wq = set ? wb[m][h].z : wb[m][h].x;
                const uint32_t wq8 = set ? wb[m][h].w : wb[m][h].y;
                mma_m16n8k16(acc[m], code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                mma_m16n8k16(acc[m], code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
            }
        }
#pragma unroll
    for (int m = 0; m < 2; ++m) {
        const __half2 sc = *reinterpret_cast<const __half2*>(&sb[m]);
        tot[m][0] = fmaf(__low2float(sc), acc[m][0] + adj, tot[m][0]);
        tot[m][1] = fmaf(__high2float(sc), acc[m][2] + adj, tot[m][1]);
    }
}

}  // namespace exmoe
