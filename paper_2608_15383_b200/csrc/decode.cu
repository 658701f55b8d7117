// Small-M grouped W4A16 kernels (decode and batched decode): fused gate/up projection + SwiGLU, and
// down projection x routing weight (the two grouped GEMMs per wave of Section 3.4; Eq. 2), plus the
// fixed-order combine.
//
// Both GEMM kernels are HBM-bound streams over the packed expert bytes.  A CTA of 8 warps owns
// `PP` 16-row panels (gate/up: panel pairs) of one active expert and splits K over `KS` warps per
// panel; each warp issues ALL of its 128-bit weight loads up front (NB blocks x 2 halves per
// matrix: up to 8 KB in flight per warp), stages the group's activation rows in shared memory while
// they fly, then dequantises in registers (shift + lop3 + one packed subtract per code pair) straight
// into m16n8k16 fragments: the packed layout IS the fragment order, so no shuffle or shared-memory
// round trip touches the weights.  Per 128-wide group the integer-valued partial sums are scaled
// in binary32 by the FP16 group scale (post-scaling: codes and activations enter the MMA exactly).
// K-split partials are reduced through shared memory in a fixed order.
#include "common.cuh"

namespace exmoe {

namespace {

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
__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two offset-binary nibbles (bits s..s+3 of each 16-bit half) -> bf16x2 of the signed codes:
// 0x4300 | u is BF16 128+u exactly; subtracting 136 leaves q = u - 8.
__device__ __forceinline__ uint32_t dequant_pair(uint32_t w, int s) {
    uint32_t v = ((w >> s) & 0x000f000fu) | 0x43004300u;
    uint32_t bias = 0x43084308u;                         // BF16 136.0 twice
    __nv_bfloat162 r = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&v), *reinterpret_cast<__nv_bfloat162*>(&bias));
    return *reinterpret_cast<uint32_t*>(&r);
}

// NB  = 128-wide blocks held in registers per warp and matrix
// NCH = 8-row activation chunks per pass (rows per pass = 8*NCH)
template <int NB, int NCH, bool GATEUP>
__global__ void __launch_bounds__(256)
decode_gemm_kernel(GemmArgs a, const __nv_bfloat16* __restrict__ x_src, __nv_bfloat16* __restrict__ act_out,
                   const float* __restrict__ topk_w, float* __restrict__ y_out, int KS, int blocks_per_warp) {
    constexpr int NM = GATEUP ? 2 : 1;
    extern __shared__ __align__(16) unsigned char smem[];
    const int K = GATEUP ? a.H : a.I;                  // reduction length
    const int NR = GATEUP ? a.I : a.H;                 // output rows of the weight matrix
    const int KB = K / kGroup;
    const int PP = 8 / KS;
    const int tiles = NR / (kPanelRows * PP);
    const int x_stride = K * 2 + 64;                   // bytes; +64 keeps 128-bit fragment loads conflict-free
    unsigned char* xs = smem;
    float* red = reinterpret_cast<float*>(smem + (size_t)8 * NCH * x_stride);   // [KS-1][PP][NM][NCH][32][4]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int ks = warp % KS, pp = warp / KS;
    const int g0 = a.wave_start[0], g1 = a.wave_start[1];
    const int n_items = (g1 - g0) * tiles;
    const size_t w13_bytes = matrix_bytes(2 * a.I, a.H);
    const bool single_chunk = (blocks_per_warp == NB);

    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int key = a.group_keys[g0 + item / tiles];
        const int tile = item % tiles;
        const int slot = key % a.num_slots;
        const int m_rows = a.counts[key], row0 = a.offsets[key];
        const uint8_t* wbase = a.slots + (size_t)slot * a.slot_stride + (GATEUP ? 0 : w13_bytes);
        const int panel = tile * PP + pp;              // panel (pair) index inside the matrix
        const uint8_t* mat[NM];
#pragma unroll
        for (int m = 0; m < NM; ++m)
            mat[m] = wbase + (size_t)((GATEUP ? 2 * panel + m : panel)) * KB * kBlockBytes;

        uint4 wreg[NM][NB][2];
        uint32_t sreg[NM][NB];

        for (int pass0 = 0; pass0 < m_rows; pass0 += 8 * NCH) {
            float tot[NM][NCH][4];
#pragma unroll
            for (int m = 0; m < NM; ++m)
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                    for (int i = 0; i < 4; ++i) tot[m][ch][i] = 0.f;

            for (int b0 = 0; b0 < blocks_per_warp; b0 += NB) {
                const int kb0 = ks * blocks_per_warp + b0;
                if (!single_chunk || pass0 == 0) {     // weights stay in registers across passes when they fit
#pragma unroll
                    for (int m = 0; m < NM; ++m)
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            const uint8_t* blk = mat[m] + (size_t)(kb0 + b) * kBlockBytes;
                            wreg[m][b][0] = ldg_stream128(blk + lane * 16);
                            wreg[m][b][1] = ldg_stream128(blk + 512 + lane * 16);
                            sreg[m][b] = ldg_stream32(blk + kCodeBytes + q * 4);
                        }
                }
                if (b0 == 0) {
                    // stage this pass's activation rows (zero rows beyond the group) while the weights fly
                    __syncthreads();                   // previous readers of xs / red are done
                    const int chunks_per_row = K / 8;
                    for (int idx = tid; idx < 8 * NCH * chunks_per_row; idx += 256) {
                        const int n = idx / chunks_per_row, ck = idx % chunks_per_row;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (pass0 + n < m_rows) {
                            const int r = row0 + pass0 + n;
                            const size_t src_row = GATEUP ? (size_t)(a.perm[r] / a.top_k) : (size_t)r;
                            v = *reinterpret_cast<const uint4*>(x_src + src_row * K + ck * 8);
                        }
                        *reinterpret_cast<uint4*>(xs + (size_t)n * x_stride + ck * 16) = v;
                    }
                    __syncthreads();
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    float acc[NM][NCH][4];
#pragma unroll
                    for (int m = 0; m < NM; ++m)
#pragma unroll
                        for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                            for (int i = 0; i < 4; ++i) acc[m][ch][i] = 0.f;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int set = 0; set < 2; ++set) {
                            const int k0 = (kb0 + b) * kGroup + 64 * h + 32 * set + 8 * c;
                            uint4 xb[NCH];
#pragma unroll
                            for (int ch = 0; ch < NCH; ++ch)
                                xb[ch] = *reinterpret_cast<const uint4*>(xs + (size_t)(8 * ch + q) * x_stride + k0 * 2);
#pragma unroll
                            for (int m = 0; m < NM; ++m) {
                                const uint32_t wq = set ? wreg[m][b][h].z : wreg[m][b][h].x;    // row q
                                const uint32_t wq8 = set ? wreg[m][b][h].w : wreg[m][b][h].y;   // row q + 8
                                uint32_t a0 = dequant_pair(wq, 0), a1 = dequant_pair(wq8, 0);
                                uint32_t a2 = dequant_pair(wq, 4), a3 = dequant_pair(wq8, 4);
#pragma unroll
                                for (int ch = 0; ch < NCH; ++ch) mma_m16n8k16(acc[m][ch], a0, a1, a2, a3, xb[ch].x, xb[ch].y);
                                a0 = dequant_pair(wq, 8), a1 = dequant_pair(wq8, 8);
                                a2 = dequant_pair(wq, 12), a3 = dequant_pair(wq8, 12);
#pragma unroll
                                for (int ch = 0; ch < NCH; ++ch) mma_m16n8k16(acc[m][ch], a0, a1, a2, a3, xb[ch].z, xb[ch].w);
                            }
                        }
                    }
#pragma unroll
                    for (int m = 0; m < NM; ++m) {     // post-scale the group's integer-valued sums
                        const __half2 sc = *reinterpret_cast<const __half2*>(&sreg[m][b]);
                        const float s_lo = __low2float(sc), s_hi = __high2float(sc);
#pragma unroll
                        for (int ch = 0; ch < NCH; ++ch) {
                            tot[m][ch][0] = fmaf(s_lo, acc[m][ch][0], tot[m][ch][0]);
                            tot[m][ch][1] = fmaf(s_lo, acc[m][ch][1], tot[m][ch][1]);
                            tot[m][ch][2] = fmaf(s_hi, acc[m][ch][2], tot[m][ch][2]);
                            tot[m][ch][3] = fmaf(s_hi, acc[m][ch][3], tot[m][ch][3]);
                        }
                    }
                }
            }

            // K-split reduction in fixed order, then the epilogue on the ks == 0 warps
            if (ks > 0) {
#pragma unroll
                for (int m = 0; m < NM; ++m)
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
                        *reinterpret_cast<float4*>(red + ((((size_t)(ks - 1) * PP + pp) * NM + m) * NCH + ch) * 128 + lane * 4) =
                            make_float4(tot[m][ch][0], tot[m][ch][1], tot[m][ch][2], tot[m][ch][3]);
            }
            __syncthreads();
            if (ks == 0) {
                for (int s = 1; s < KS; ++s)
#pragma unroll
                    for (int m = 0; m < NM; ++m)
#pragma unroll
                        for (int ch = 0; ch < NCH; ++ch) {
                            const float4 v = *reinterpret_cast<const float4*>(
                                red + ((((size_t)(s - 1) * PP + pp) * NM + m) * NCH + ch) * 128 + lane * 4);
                            tot[m][ch][0] += v.x; tot[m][ch][1] += v.y; tot[m][ch][2] += v.z; tot[m][ch][3] += v.w;
                        }
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int n = pass0 + 8 * ch + 2 * c + (i & 1);
                        if (n >= m_rows) continue;
                        const int r = row0 + n;
                        const int orow = (tile * PP + pp) * kPanelRows + q + 8 * (i >> 1);
                        if (GATEUP) {
                            const float g = tot[0][ch][i], u = tot[NM - 1][ch][i];
                            const float act = g / (1.f + __expf(-g)) * u;
                            act_out[(size_t)r * a.I + orow] = __float2bfloat16_rn(act);
                        } else {
                            const int pair = a.perm[r];
                            y_out[(size_t)pair * a.H + orow] = topk_w[pair] * tot[0][ch][i];
                        }
                    }
            }
        }
    }
}

// K split over KS warps (KS in {1,2,4,8}, 8/KS panels per CTA) and register depth NB; aims at
// four blocks per warp so that all of a warp's weights are in flight at once.
struct DecodeCfg { int NB, KS, bpw; };
DecodeCfg pick_cfg(int K, int rows) {
    const int KB = K / kGroup;
    int pref = 1;
    while (pref < 8 && KB / (pref * 2) >= 4) pref *= 2;
    const int order[4][4] = {{1, 2, 4, 8}, {2, 1, 4, 8}, {4, 2, 8, 1}, {8, 4, 2, 1}};
    const int* cand = order[pref == 1 ? 0 : pref == 2 ? 1 : pref == 4 ? 2 : 3];
    for (int i = 0; i < 4; ++i) {
        const int ksv = cand[i];
        if (KB % ksv || rows % (kPanelRows * (8 / ksv))) continue;
        const int bpw = KB / ksv;
        return {(bpw % 4 == 0) ? 4 : (bpw % 2 == 0) ? 2 : 1, ksv, bpw};
    }
    return {1, 1, KB};                                  // rows % 128 == 0 always makes KS = 1 feasible
}

template <int NB, int NCH, bool GATEUP>
void launch_cfg(const GemmArgs& a, const __nv_bfloat16* x, __nv_bfloat16* act, const float* w, float* y,
                const DecodeCfg& cfg, int max_groups, cudaStream_t st) {
    constexpr int NM = GATEUP ? 2 : 1;
    const int K = GATEUP ? a.H : a.I, NR = GATEUP ? a.I : a.H;
    const int PP = 8 / cfg.KS;
    const int tiles = NR / (kPanelRows * PP);
    const size_t smem = (size_t)8 * NCH * (K * 2 + 64) + (size_t)(cfg.KS - 1) * PP * NM * NCH * 128 * 4;
    auto kern = decode_gemm_kernel<NB, NCH, GATEUP>;
    static bool attr_done = false;                      // per instantiation
    if (!attr_done) {
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        attr_done = true;
    }
    long long items = (long long)max_groups * tiles;
    const int grid = (int)(items < 148 * 8 ? (items < 1 ? 1 : items) : 148 * 8);
    kern<<<grid, 256, smem, st>>>(a, x, act, w, y, cfg.KS, cfg.bpw);
    count_launch();
}

template <bool GATEUP>
void launch_decode(const GemmArgs& a, const __nv_bfloat16* x, __nv_bfloat16* act, const float* w, float* y,
                   int max_rows, int max_groups, cudaStream_t st) {
    const int K = GATEUP ? a.H : a.I, NR = GATEUP ? a.I : a.H;
    const DecodeCfg cfg = pick_cfg(K, NR);
    // rows per pass: one 8-row chunk covers decode; more chunks amortise the dequantisation
    int nch = max_rows <= 8 ? 1 : (max_rows <= 16 ? 2 : 4);
    while (nch > 1 && (size_t)8 * nch * (K * 2 + 64) > 150 * 1024) nch >>= 1;
#define EXMOE_DISPATCH(NBv)                                                                     \
    if (nch == 1) launch_cfg<NBv, 1, GATEUP>(a, x, act, w, y, cfg, max_groups, st);             \
    else if (nch == 2) launch_cfg<NBv, 2, GATEUP>(a, x, act, w, y, cfg, max_groups, st);        \
    else launch_cfg<NBv, 4, GATEUP>(a, x, act, w, y, cfg, max_groups, st);
    if (cfg.NB == 4) { EXMOE_DISPATCH(4) }
    else if (cfg.NB == 2) { EXMOE_DISPATCH(2) }
    else { EXMOE_DISPATCH(1) }
#undef EXMOE_DISPATCH
}

// out[t] = bf16( sum_{j=0..k-1} Y[t*k + j] ), binary32, fixed order; pairs with an invalid id add nothing
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ y, const int32_t* __restrict__ ids, int E, int T, int k, int H,
               __nv_bfloat16* __restrict__ out) {
    const int per_row = H / 4;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)T * per_row) return;
    const int t = (int)(idx / per_row), h4 = (int)(idx % per_row);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = 0; j < k; ++j) {
        const int id = ids[t * k + j];
        if (id < 0 || id >= E) continue;
        const float4 v = *reinterpret_cast<const float4*>(y + ((size_t)t * k + j) * H + h4 * 4);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t*>(&lo);
    o.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + (size_t)t * H + h4 * 4) = o;
}

}  // namespace

void launch_decode_gateup(const GemmArgs& a, const __nv_bfloat16* hidden, __nv_bfloat16* act, int max_rows,
                          int max_groups, cudaStream_t st) {
    launch_decode<true>(a, hidden, act, nullptr, nullptr, max_rows, max_groups, st);
}
void launch_decode_down(const GemmArgs& a, const __nv_bfloat16* act, const float* topk_w, float* y, int max_rows,
                        int max_groups, cudaStream_t st) {
    launch_decode<false>(a, act, nullptr, topk_w, y, max_rows, max_groups, st);
}
void launch_combine(const float* y, const int32_t* ids, int E, int T, int k, int H, __nv_bfloat16* out,
                    cudaStream_t st) {
    const long long n = (long long)T * (H / 4);
    combine_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(y, ids, E, T, k, H, out);
    count_launch();
}

}  // namespace exmoe
