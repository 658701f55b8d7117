// Small-M grouped W4A16 kernels (decode and batched decode): fused gate/up projection + SwiGLU, and
// down projection x routing weight (the two grouped GEMMs per wave of Section 3.4; Eq. 2), plus the
// fixed-order combine.
//
// Both GEMM kernels are HBM-bound streams over the packed expert bytes.  A CTA of 8 warps owns
// `PP` 16-row panels (gate/up: panel pairs) of one active expert and splits K over `KS` warps per
// panel; each warp issues ALL of its 128-bit weight loads up front (NB blocks x 2 halves per
// matrix: up to 8 KB in flight per warp), stages the group's activation rows in shared memory while
// they fly, then dequantises in registers (one shift and one lop3 per code pair; the code bias of 136 is
// removed after the MMA with a per-block correction formed while the activations are staged) straight
// into m16n8k16 fragments: the packed layout IS the fragment order, so no shuffle or shared-memory
// round trip touches the weights.  Per 128-wide group the integer-valued partial sums are scaled
// in binary32 by the FP16 group scale (post-scaling: codes and activations enter the MMA exactly).
// K-split partials are reduced through shared memory in a fixed order.
//
// Two flavours share the body:
//   SMALL (T*k <= kSmallMaxPairs): a decode step is launch-latency bound, so the chain of dependent global
//     loads is cut to two levels: every CTA rebuilds the wave's token grouping (histogram, prefix
//     sum, stable permutation) in shared memory straight from topk_ids; CTA 0 also publishes it.
//     The down kernel is launched with programmatic dependent launch: it prefetches its weights
//     while the gate/up kernel still runs, and it folds the fixed-order combine in: the last CTA
//     to finish a (token, column tile) sums the k pair rows in order j = 0..k-1 (no spin wait).
//   PAIR (same sizes, one wave; the allocation-free entry point up to kPairMaxPairs): no grouping at all; see
//     pair_gateup_kernel, token_down_kernel (one token) and token_down_bulk_kernel (two or more tokens).
// Larger batches run on the streaming kernels (stream.cu) or the tensor-core kernels (prefill.cu) with the
// grouping kernels' global plan and the separate combine kernel defined here.
#include "common.cuh"
#include "frag.cuh"
#include "mbar.cuh"

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
// loads that must be ISSUED where they are written (volatile asm: the compiler may not sink them to their use)
__device__ __forceinline__ uint4 ldg_early128(const void* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float ldg_early_f32(const void* p) {
    float v;
    asm volatile("ld.global.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
// Shared-memory plan of ONE wave, rebuilt by every CTA of the SMALL kernels.
struct SmallPlan {
    int* cnt;     // [C] pairs per slot in this wave
    int* off;     // [C + 1] exclusive prefix sum (rows local to the wave)
    int* gkeys;   // [C] slots with cnt > 0, ascending
    int* lkey;    // [P] slot of the pair in this wave, -1 other wave, -2 invalid id
    int* perm;    // [P] pair indices of this wave ordered by (slot, pair)
    int n_groups;
    int row_base; // valid pairs in earlier waves = first grouped row of this wave
};

struct SmallArgs {
    const int32_t* ids;
    const int32_t* wave_of;   // null in identity mode (C = E: slot = expert id, one wave)
    const int32_t* slot_of;
    int n_pairs, E, wave;
    int32_t* pub_counts;      // global plan arrays published by CTA 0 of the gate/up kernel
    int32_t* pub_offsets;
    int32_t* pub_perm;
    int32_t* header;
    int* status;
    int* arrive;              // [T * tiles] arrival counters of the fused combine (zero between calls)
    __nv_bfloat16* out;       // [T, H]
    int32_t* saved_ids;       // [kPairMaxPairs] copy of the ids kept by the pairwise path
};

__device__ __forceinline__ void build_small_plan(const SmallArgs& sa, int C, SmallPlan& sp, int* s_scalars) {
    const int tid = threadIdx.x, P = sa.n_pairs;
    for (int i = tid; i < C; i += blockDim.x) sp.cnt[i] = 0;
    if (tid < 4) s_scalars[tid] = 0;                      // [0] rows before this wave, [1] n_groups, [2] bad id
    __syncthreads();
    for (int p = tid; p < P; p += blockDim.x) {
        const int id = sa.ids[p];
        int lk = -2;
        if (id >= 0 && id < sa.E) {
            const int w = sa.wave_of ? sa.wave_of[id] : 0;
            const int s = sa.slot_of ? sa.slot_of[id] : id;
            if (w < sa.wave) atomicAdd(&s_scalars[0], 1);
            lk = (w == sa.wave) ? s : -1;
            if (lk >= 0) atomicAdd(&sp.cnt[lk], 1);
        } else {
            s_scalars[2] = 1;
        }
        sp.lkey[p] = lk;
    }
    __syncthreads();
    if (tid < 32) {
        const unsigned lt = (1u << tid) - 1u;
        int running = 0, ng = 0;
        for (int base = 0; base < C; base += 32) {
            const int kx = base + tid;
            const int v = kx < C ? sp.cnt[kx] : 0;
            int incl = v;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, d);
                if (tid >= d) incl += o;
            }
            if (kx < C) sp.off[kx] = running + incl - v;
            const unsigned b = __ballot_sync(0xffffffffu, v > 0);
            if (v > 0) sp.gkeys[ng + __popc(b & lt)] = kx;
            ng += __popc(b);
            running += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (tid == 0) {
            sp.off[C] = running;
            s_scalars[1] = ng;
        }
    }
    __syncthreads();
    for (int p = tid; p < P; p += blockDim.x) {
        const int lk = sp.lkey[p];
        if (lk < 0) continue;
        int r = 0;
        for (int j = 0; j < p; ++j) r += (sp.lkey[j] == lk);
        sp.perm[sp.off[lk] + r] = p;
    }
    __syncthreads();
    sp.row_base = s_scalars[0];
    sp.n_groups = s_scalars[1];
}

// NB  = 128-wide blocks held in registers per warp and matrix
// NCH = 8-row activation chunks per pass (rows per pass = 8*NCH)
enum { MODE_SMALL = 1, MODE_PAIR = 2 };

// MODE_SMALL : every CTA rebuilds the wave's grouping in shared memory (T*k <= kSmallMaxPairs)
// MODE_PAIR  : one item per token-expert pair, no grouping at all (T*k <= 32, gate/up only)
template <int NB, int NCH, bool GATEUP, int MODE>
__global__ void __launch_bounds__(256, 1)
decode_gemm_kernel(GemmArgs a, SmallArgs sa, const __nv_bfloat16* __restrict__ x_src,
                   __nv_bfloat16* __restrict__ act_out, const float* __restrict__ topk_w, float* __restrict__ y_out,
                   int KS, int blocks_per_warp) {
    constexpr int NM = GATEUP ? 2 : 1;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_scalars[4];
    const int K = GATEUP ? a.H : a.I;                  // reduction length
    const int NR = GATEUP ? a.I : a.H;                 // output rows of the weight matrix
    const int KB = K / kGroup;
    const int PP = 8 / KS;
    const int tiles = NR / (kPanelRows * PP);
    const int x_stride = K * 2 + 64;                   // bytes; +64 keeps 128-bit fragment loads conflict-free
    unsigned char* xs = smem;
    float* red = reinterpret_cast<float*>(smem + (size_t)8 * NCH * x_stride);   // [KS-1][PP][NM][NCH][32][4]
    float* adj = red + (size_t)(KS - 1) * PP * NM * NCH * 128;                  // [KB][8*NCH]
    int* plan_mem = reinterpret_cast<int*>(adj + (size_t)KB * 8 * NCH);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int ks = warp % KS, pp = warp / KS;
    const size_t w13_bytes = matrix_bytes(2 * a.I, a.H);
    const bool single_chunk = (blocks_per_warp == NB);
    const int C = a.num_slots;

    constexpr bool SMALL = (MODE == MODE_SMALL);
    constexpr bool PAIR = (MODE == MODE_PAIR);
    SmallPlan sp{};
    int n_items;
    if (PAIR) {
        grid_launch_dependents();
        n_items = sa.n_pairs * tiles;
        if (blockIdx.x == 0 && tid < sa.n_pairs) {     // keep the ids so the plan can be materialised on request
            const int id = sa.ids[tid];
            sa.saved_ids[tid] = id;
            if (id < 0 || id >= sa.E) atomicExch(sa.status, EXMOE_ERR_BAD_EXPERT_ID);
        }
    } else {
        if (GATEUP) grid_launch_dependents();          // let the down kernel start prefetching its weights
        sp.cnt = plan_mem;
        sp.off = sp.cnt + C;
        sp.gkeys = sp.off + C + 1;
        sp.lkey = sp.gkeys + C;
        sp.perm = sp.lkey + sa.n_pairs;
        build_small_plan(sa, C, sp, s_scalars);
        n_items = sp.n_groups * tiles;
        if (GATEUP && blockIdx.x == 0) {               // publish the wave's part of the plan (test hook, stats)
            for (int i = tid; i < C; i += 256) {
                sa.pub_counts[sa.wave * C + i] = sp.cnt[i];
                sa.pub_offsets[sa.wave * C + i] = sp.row_base + sp.off[i];
            }
            for (int i = tid; i < sp.off[C]; i += 256) sa.pub_perm[sp.row_base + i] = sp.perm[i];
            if (tid == 0) {
                sa.pub_offsets[sa.wave * C + C] = sp.row_base + sp.off[C];
                if (!sa.wave_of) {                     // identity mode: no resolution kernel wrote the header
                    sa.header[HDR_N_ACTIVE] = sp.n_groups;
                    sa.header[HDR_N_WAVES] = sp.n_groups ? 1 : 0;
                    sa.header[HDR_N_MISSES] = 0;
                    sa.header[HDR_BAD_ID] = s_scalars[2];
                }
                if (s_scalars[2]) atomicExch(sa.status, EXMOE_ERR_BAD_EXPERT_ID);
            }
        }
    }

    bool waited = false;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int tile = item % tiles;
        int slot, m_rows, row0, lrow0 = 0;
        if (PAIR) {
            const int p = item / tiles;                // activation row = pair index, one row per item
            const int id = sa.ids[p];
            if (id < 0 || id >= sa.E) continue;        // uniform over the CTA
            slot = sa.slot_of ? sa.slot_of[id] : id;
            m_rows = 1;
            row0 = p;
        } else {
            slot = sp.gkeys[item / tiles];
            m_rows = sp.cnt[slot];
            lrow0 = sp.off[slot];
            row0 = sp.row_base + lrow0;
        }
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
                    if (SMALL && !GATEUP && !waited) {
                        grid_dependency_wait();        // the gate/up kernel's activations are complete and visible
                        waited = true;
                    }
                    __syncthreads();                   // previous readers of xs / red are done
                    // also: adj[kb][n] = -136 * sum_k x[n][k] over each 128-wide block (see the block loop)
                    const int chunks_per_row = K / 8;
                    const int rows_here = min(8 * NCH, m_rows - pass0);   // rows beyond are zero registers, not staged
                    const int total = rows_here * chunks_per_row;
                    for (int base = warp * 32; base < total; base += 256) {
                        const int idx = base + lane;
                        const int n = idx / chunks_per_row, ck = idx % chunks_per_row;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (idx < total) {
                            size_t src_row;
                            if (PAIR) src_row = (size_t)(row0 / a.top_k);
                            else if (GATEUP) src_row = (size_t)(sp.perm[lrow0 + pass0 + n] / a.top_k);
                            else src_row = (size_t)(row0 + pass0 + n);
                            v = *reinterpret_cast<const uint4*>(x_src + src_row * K + ck * 8);
                            *reinterpret_cast<uint4*>(xs + (size_t)n * x_stride + ck * 16) = v;
                        }
                        float sx = sum8_bf16(v);
#pragma unroll
                        for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);   // 16 chunks = one block
                        if (idx < total && (ck & 15) == 0) adj[(ck >> 4) * (8 * NCH) + n] = -136.f * sx;
                    }
                    __syncthreads();
                }
                const int rows_here = min(8 * NCH, m_rows - pass0);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    // acc = sum (136 + q) x over the block's 128 columns (codes enter the MMA as 128 + u,
                    // exact in BF16); adj = -136 * sum x was formed while staging; acc + adj = sum q x.
                    float acc[NM][NCH][4];
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int m = 0; m < NM; ++m) acc[m][ch][i] = 0.f;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int set = 0; set < 2; ++set) {
                            const int k0 = (kb0 + b) * kGroup + 64 * h + 32 * set + 8 * c;
                            uint4 xb[NCH];
#pragma unroll
                            for (int ch = 0; ch < NCH; ++ch) {
                                xb[ch] = make_uint4(0, 0, 0, 0);
                                if (8 * ch + q < rows_here)
                                    xb[ch] = *reinterpret_cast<const uint4*>(xs + (size_t)(8 * ch + q) * x_stride + k0 * 2);
                            }
#pragma unroll
                            for (int m = 0; m < NM; ++m) {
                                const uint32_t wq = set ? wreg[m][b][h].z : wreg[m][b][h].x;    // row q
                                const uint32_t wq8 = set ? wreg[m][b][h].w : wreg[m][b][h].y;   // row q + 8
                                uint32_t a0 = code_pair(wq, 0), a1 = code_pair(wq8, 0);
                                uint32_t a2 = code_pair(wq, 4), a3 = code_pair(wq8, 4);
#pragma unroll
                                for (int ch = 0; ch < NCH; ++ch) mma_m16n8k16(acc[m][ch], a0, a1, a2, a3, xb[ch].x, xb[ch].y);
                                a0 = code_pair(wq, 8), a1 = code_pair(wq8, 8);
                                a2 = code_pair(wq, 12), a3 = code_pair(wq8, 12);
#pragma unroll
                                for (int ch = 0; ch < NCH; ++ch) mma_m16n8k16(acc[m][ch], a0, a1, a2, a3, xb[ch].z, xb[ch].w);
                            }
                        }
                    }
                    float2 cr[NCH];
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
                        cr[ch] = *reinterpret_cast<const float2*>(adj + (size_t)(kb0 + b) * (8 * NCH) + 8 * ch + 2 * c);
#pragma unroll
                    for (int m = 0; m < NM; ++m) {     // post-scale the group's integer-valued sums
                        const __half2 sc = *reinterpret_cast<const __half2*>(&sreg[m][b]);
                        const float s_lo = __low2float(sc), s_hi = __high2float(sc);
#pragma unroll
                        for (int ch = 0; ch < NCH; ++ch) {
                            tot[m][ch][0] = fmaf(s_lo, acc[m][ch][0] + cr[ch].x, tot[m][ch][0]);
                            tot[m][ch][1] = fmaf(s_lo, acc[m][ch][1] + cr[ch].y, tot[m][ch][1]);
                            tot[m][ch][2] = fmaf(s_hi, acc[m][ch][2] + cr[ch].x, tot[m][ch][2]);
                            tot[m][ch][3] = fmaf(s_hi, acc[m][ch][3] + cr[ch].y, tot[m][ch][3]);
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
                        const int orow = (tile * PP + pp) * kPanelRows + q + 8 * (i >> 1);
                        if (GATEUP) {
                            const float g = tot[0][ch][i], u = tot[NM - 1][ch][i];
                            const float act = g / (1.f + __expf(-g)) * u;
                            act_out[(size_t)(row0 + n) * a.I + orow] = __float2bfloat16_rn(act);
                        } else {
                            const int pair = sp.perm[lrow0 + n];
                            y_out[(size_t)pair * a.H + orow] = topk_w[pair] * tot[0][ch][i];
                        }
                    }
            }
        }

        if (SMALL && !GATEUP) {
            // Fused combine (Eq. 2's sum over the selected experts): the CTA that completes the last
            // pair of a token for this column tile adds the k rows in the fixed order j = 0..k-1.
            const int cols = kPanelRows * PP, col0 = tile * cols, k = a.top_k;
            __threadfence();
            __syncthreads();
            for (int i = 0; i < m_rows; ++i) {
                const int t = sp.perm[lrow0 + i] / k;
                __shared__ int s_last;
                if (tid == 0) {
                    int need = 0;
                    for (int j = 0; j < k; ++j) need += (sp.lkey[t * k + j] != -2);
                    const int old = atomicAdd(&sa.arrive[t * tiles + tile], 1);
                    s_last = (old == need - 1);
                    if (s_last) sa.arrive[t * tiles + tile] = 0;          // self-cleaning for the next call
                }
                __syncthreads();
                if (s_last) {
                    __threadfence();
                    for (int col = tid; col < cols; col += 256) {
                        float sum = 0.f;
                        for (int j = 0; j < k; ++j)
                            if (sp.lkey[t * k + j] != -2) sum += __ldcg(y_out + (size_t)(t * k + j) * a.H + col0 + col);
                        sa.out[(size_t)t * a.H + col0 + col] = __float2bfloat16_rn(sum);
                    }
                }
                __syncthreads();
            }
        }
    }
    if (SMALL && !GATEUP && !waited) grid_dependency_wait();
    if (SMALL && GATEUP && blockIdx.x == 0) {
        // tokens whose ids are all invalid get no contribution: their output row is zero
        const int k = a.top_k, T = sa.n_pairs / k;
        if (sa.wave == 0 && s_scalars[2])
            for (int t = 0; t < T; ++t) {
                int need = 0;
                for (int j = 0; j < k; ++j) need += (sp.lkey[t * k + j] != -2);
                if (need == 0)
                    for (int col = tid; col < a.H; col += 256) sa.out[(size_t)t * a.H + col] = __float2bfloat16_rn(0.f);
            }
    }
}


// Down projection + routing weight + combine for tiny batches (T*k <= 32, one wave): one CTA per
// (token, 16-column panel), one warp per selected expert.  Each warp streams its expert's panel over
// the whole K (all loads in flight at once), the k results are summed in the fixed order j = 0..k-1
// through shared memory and the BF16 output row is written directly: no pair buffer, no atomics.
// Launched as a programmatic dependent of the gate/up kernel: weights are prefetched before the
// dependency wait.  `KSg`/`bpwg` replay the grouped kernel's K-split order so that both paths round
// identically.
// Placement matters at one token: with its 139 registers a CTA of this kernel does not fit beside a gate/up CTA
// that is still running, so it starts on SMs the gate/up kernel has left.  Two variants that did fit (a 128-register
// cap; a prologue without integer divisions, which the compiler allocated in 128 registers) started their weight
// loads on the 40 SMs holding a single gate/up CTA, delayed the kernel they then wait for, and measured 14.2 and
// 13.9 us per step against 12.65; forcing the separation with a 220 KB shared-memory request instead cost a
// carve-out change per launch (13.7 us).  Re-time the whole step, not the kernel alone, after touching this kernel.
#ifndef EXMOE_DOWN_ABLATE
#define EXMOE_DOWN_ABLATE 0
#endif
template <int NBT>
__global__ void __launch_bounds__(256)
token_down_kernel(GemmArgs a, SmallArgs sa, const __nv_bfloat16* __restrict__ act, const float* __restrict__ topk_w,
                  int bpwg) {
    extern __shared__ __align__(128) unsigned char smem[];
    grid_launch_dependents();                          // the next kernel in the stream may be placed (it waits for this one)
    const int K = a.I, KB = K / kGroup, k = a.top_k;
    const int x_stride = K * 2 + 64;
    unsigned char* xs = smem;                                          // [k][x_stride]
    float* ys = reinterpret_cast<float*>(smem + (size_t)k * x_stride); // [k][16]
    int* s_valid = reinterpret_cast<int*>(ys + k * 16);                // [k]
    float* adj = reinterpret_cast<float*>(s_valid + k);                // [KB][k]  -136 * block sums of the activations
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int panels = a.H / kPanelRows;
    const int t = blockIdx.x / panels, panel = blockIdx.x % panels;
    const size_t w13_bytes = matrix_bytes(2 * a.I, a.H);
    bool staged = false;

    for (int j0 = 0; j0 < k; j0 += 8) {
        const int j = j0 + warp;
        const int pair = t * k + j;
        int id = -1;
        if (j < k) id = sa.ids[pair];
        const bool valid = (j < k) && id >= 0 && id < sa.E;
        const float rw = valid ? ldg_early_f32(topk_w + pair) : 0.f;   // requested early: needed only in the epilogue
        float result[2] = {0.f, 0.f};
        float total[2] = {0.f, 0.f};
        for (int b0 = 0; b0 < KB; b0 += NBT) {
            uint4 wreg[NBT][2];
            uint32_t sreg[NBT];
            if (valid) {
                const int slot = sa.slot_of ? sa.slot_of[id] : id;
                const uint8_t* mat = a.slots + (size_t)slot * a.slot_stride + w13_bytes + (size_t)panel * KB * kBlockBytes;
#pragma unroll
                for (int b = 0; b < NBT; ++b) {
                    const uint8_t* blk = mat + (size_t)(b0 + b) * kBlockBytes;
                    wreg[b][0] = ldg_stream128(blk + lane * 16);
                    wreg[b][1] = ldg_stream128(blk + 512 + lane * 16);
                    sreg[b] = ldg_stream32(blk + kCodeBytes + q * 4);
                }
            }
            if (b0 == 0) {                          // first chunk: the activations arrive after the weights were requested
                if (!staged) grid_dependency_wait();
                staged = true;
#if EXMOE_DOWN_ABLATE == 1
                if (wreg[0][0].x == 0x12345u && sreg[0] == 7u) sa.out[0] = __float2bfloat16_rn(1.f);
                return;                             // timing only: weights requested, dependency met
#endif
                // Every warp stages the ONE activation row its expert needs (row j of the token) and forms that row's block
                // sums itself: all of its 16-byte chunks in flight at once (one L2 round trip), no CTA-wide barrier before
                // the arithmetic.  Chunk -> lane mapping and butterfly as in the other staging loops: same bits.
                if (j < k) {
                    const int chunks_per_row = K / 8;
                    const uint4* src = reinterpret_cast<const uint4*>(act + (size_t)(t * k + j) * K);
                    for (int base0 = 0; base0 < chunks_per_row; base0 += 4 * 32) {
                        uint4 v[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int ck = base0 + u * 32 + lane;
                            v[u] = make_uint4(0, 0, 0, 0);
                            if (ck < chunks_per_row) v[u] = __ldcg(src + ck);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int ck = base0 + u * 32 + lane;
                            if (ck < chunks_per_row) *reinterpret_cast<uint4*>(xs + (size_t)j * x_stride + ck * 16) = v[u];
                            float sx = sum8_bf16(v[u]);
#pragma unroll
                            for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
                            if (ck < chunks_per_row && (ck & 15) == 0) adj[(ck >> 4) * k + j] = -136.f * sx;
                        }
                    }
                }
                __syncwarp();
#if EXMOE_DOWN_ABLATE == 2
                if (wreg[0][0].x == 0x12345u && sreg[0] == 7u) sa.out[0] = __float2bfloat16_rn(1.f);
                return;                             // timing only: ... and activations staged
#endif
            }
            if (valid) {
#pragma unroll
                for (int b = 0; b < NBT; ++b) {
                    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int set = 0; set < 2; ++set) {
                            const int k0 = (b0 + b) * kGroup + 64 * h + 32 * set + 8 * c;
                            uint4 xb = make_uint4(0, 0, 0, 0);
                            if (q == 0) xb = *reinterpret_cast<const uint4*>(xs + (size_t)j * x_stride + k0 * 2);
                            const uint32_t wq = set ? wreg[b][h].z : wreg[b][h].x;
                            const uint32_t wq8 = set ? wreg[b][h].w : wreg[b][h].y;
                            mma_m16n8k16(acc, code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                            mma_m16n8k16(acc, code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
                        }
                    const __half2 sc = *reinterpret_cast<const __half2*>(&sreg[b]);
                    const float cr = adj[(b0 + b) * k + j];
                    total[0] = fmaf(__low2float(sc), acc[0] + cr, total[0]);
                    total[1] = fmaf(__high2float(sc), acc[2] + cr, total[1]);
                    if ((b0 + b + 1) % bpwg == 0) {            // end of one K-split range of the grouped kernel
                        const bool first = (b0 + b + 1 == bpwg);
                        result[0] = first ? total[0] : result[0] + total[0];
                        result[1] = first ? total[1] : result[1] + total[1];
                        total[0] = total[1] = 0.f;
                    }
                }
            }
        }
        if (j < k) {
            if (lane == 0) s_valid[j] = valid ? 1 : 0;
            if (c == 0) {
                ys[j * 16 + q] = rw * result[0];
                ys[j * 16 + q + 8] = rw * result[1];
            }
        }
    }
    if (!staged) grid_dependency_wait();
    __syncthreads();
    if (tid < 16) {
        float sum = 0.f;
        for (int j = 0; j < k; ++j)
            if (s_valid[j]) sum += ys[j * 16 + tid];
        sa.out[(size_t)t * a.H + panel * kPanelRows + tid] = __float2bfloat16_rn(sum);
    }
}


// Gate/up + SwiGLU for tiny batches (T*k <= 32, one wave): one CTA per (token-expert pair, tile of
// 8/KS panel pairs), one activation row, every weight load of a warp issued before anything else.
// Straight-line code (no item, pass or chunk loops) so that two CTAs fit an SM and the whole grid is
// one resident wave; the arithmetic and its order are those of decode_gemm_kernel.
template <int NB>
__device__ __forceinline__ void pair_gateup_item(const GemmArgs& a, const SmallArgs& sa,
                                                 const __nv_bfloat16* __restrict__ hidden,
                                                 __nv_bfloat16* __restrict__ act_out, int ks_log2, int p, int token,
                                                 int tile, unsigned char* smem) {
    // No integer division anywhere before the first loads are issued (a runtime division is a dependent chain of
    // some 25 instructions): the K split is a power of two, pair and tile come from the grid's coordinates.
    const int K = a.H, KB = K / kGroup, KS = 1 << ks_log2, PP = 8 >> ks_log2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int ks = warp & (KS - 1), pp = warp >> ks_log2;
    unsigned char* xs = smem;                                            // one activation row
    float* red = reinterpret_cast<float*>(smem + K * 2 + 64);            // [KS-1][PP][2][32][4]
    float* adj = red + (size_t)(KS - 1) * PP * 2 * 128;                  // [KB]

    // The hidden row does not depend on the ids: request it first so that it is not queued behind the weights.
    const __nv_bfloat16* xrow = hidden + (size_t)token * K;
    uint4 xpre = make_uint4(0, 0, 0, 0);
    if (tid < K / 8) xpre = ldg_early128(xrow + tid * 8);
    const int id = sa.ids[p];
    if (id < 0 || id >= sa.E) return;                  // uniform over the CTA; the pair contributes nothing
    const int slot = sa.slot_of ? sa.slot_of[id] : id;
    const int panel = tile * PP + pp;
    const uint8_t* wbase = a.slots + (size_t)slot * a.slot_stride;
    uint4 wreg[2][NB][2];
    uint32_t sreg[2][NB];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const uint8_t* blk = wbase + ((size_t)(2 * panel + m) * KB + ks * NB + b) * kBlockBytes;
            wreg[m][b][0] = ldg_stream128(blk + lane * 16);
            wreg[m][b][1] = ldg_stream128(blk + 512 + lane * 16);
            sreg[m][b] = ldg_stream32(blk + kCodeBytes + q * 4);
        }
    // stage the token's hidden row; adj[kb] = -136 * (sum of the row over block kb)
    const int total = K / 8;
    for (int base = warp * 32; base < total; base += 256) {
        const int ck = base + lane;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (ck < total) {
            v = (base < 256) ? xpre : *reinterpret_cast<const uint4*>(xrow + ck * 8);
            *reinterpret_cast<uint4*>(xs + ck * 16) = v;
        }
        float sx = sum8_bf16(v);
#pragma unroll
        for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
        if (ck < total && (ck & 15) == 0) adj[ck >> 4] = -136.f * sx;
    }
    __syncthreads();

    float tot[2][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int i = 0; i < 4; ++i) tot[m][i] = 0.f;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        float acc[2][4];
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[m][i] = 0.f;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int set = 0; set < 2; ++set) {
                const int k0 = (ks * NB + b) * kGroup + 64 * h + 32 * set + 8 * c;
                uint4 xb = make_uint4(0, 0, 0, 0);
                if (q == 0) xb = *reinterpret_cast<const uint4*>(xs + k0 * 2);
#pragma unroll
                for (int m = 0; m < 2; ++m) {
                    const uint32_t wq = set ? wreg[m][b][h].z : wreg[m][b][h].x;
                    const uint32_t wq8 = set ? wreg[m][b][h].w : wreg[m][b][h].y;
                    mma_m16n8k16(acc[m], code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                    mma_m16n8k16(acc[m], code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
                }
            }
        const float cr = adj[ks * NB + b];             // column 0 is the only live one; others are discarded
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const __half2 sc = *reinterpret_cast<const __half2*>(&sreg[m][b]);
            const float s_lo = __low2float(sc), s_hi = __high2float(sc);
            tot[m][0] = fmaf(s_lo, acc[m][0] + cr, tot[m][0]);
            tot[m][2] = fmaf(s_hi, acc[m][2] + cr, tot[m][2]);
        }
    }
    if (ks > 0 && c == 0) {
        red[(((ks - 1) * PP + pp) * 2 + 0) * 16 + q] = tot[0][0];
        red[(((ks - 1) * PP + pp) * 2 + 0) * 16 + q + 8] = tot[0][2];
        red[(((ks - 1) * PP + pp) * 2 + 1) * 16 + q] = tot[1][0];
        red[(((ks - 1) * PP + pp) * 2 + 1) * 16 + q + 8] = tot[1][2];
    }
    __syncthreads();
    if (ks == 0 && c == 0) {
        for (int s = 1; s < KS; ++s) {
            tot[0][0] += red[(((s - 1) * PP + pp) * 2 + 0) * 16 + q];
            tot[0][2] += red[(((s - 1) * PP + pp) * 2 + 0) * 16 + q + 8];
            tot[1][0] += red[(((s - 1) * PP + pp) * 2 + 1) * 16 + q];
            tot[1][2] += red[(((s - 1) * PP + pp) * 2 + 1) * 16 + q + 8];
        }
#pragma unroll
        for (int i = 0; i < 4; i += 2) {
            const float g = tot[0][i], u = tot[1][i];
            act_out[(size_t)p * a.I + panel * kPanelRows + q + 4 * i] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * u);
        }
    }
}

// keep the ids of a pairwise call (so the plan can be materialised on request) and flag invalid ones
__device__ __forceinline__ void keep_pair_ids(const SmallArgs& sa) {
    const int tid = threadIdx.x;
    if (tid < sa.n_pairs) {
        const int v = sa.ids[tid];
        sa.saved_ids[tid] = v;
        if (v < 0 || v >= sa.E) atomicExch(sa.status, EXMOE_ERR_BAD_EXPERT_ID);
    }
}

template <int NB>
__global__ void __launch_bounds__(256, 2)
pair_gateup_kernel(GemmArgs a, SmallArgs sa, const __nv_bfloat16* __restrict__ hidden,
                   __nv_bfloat16* __restrict__ act_out, int ks_log2) {
    // grid = (tiles of the intermediate dimension, selected expert j, token t): pair p = t * k + j
    extern __shared__ __align__(128) unsigned char smem[];
    grid_dependency_wait();                            // launched as a programmatic dependent of whatever precedes it in the stream
    grid_launch_dependents();
    if ((blockIdx.x | blockIdx.y | blockIdx.z) == 0) keep_pair_ids(sa);
    pair_gateup_item<NB>(a, sa, hidden, act_out, ks_log2, (int)(blockIdx.z * a.top_k + blockIdx.y), (int)blockIdx.z,
                         (int)blockIdx.x, smem);
}

// ------------------------------------------------------------------------------------------------
// Wide variant of the per-pair gate/up kernel: ONE CTA of 16 warps per SM instead of two of 8, each warp one
// (panel pair, K range) unit held in registers, and every warp a pipeline of its own: its K range of the hidden
// row goes into a private piece of shared memory, it forms the range's block corrections itself (same chunk ->
// lane mapping and butterfly as the staging loops above: same bits), requests its blocks AHEAD blocks before it
// needs them and starts on a block as soon as that block's registers have arrived.  No CTA-wide barrier before the
// K-range partials meet, so the conversion of the early blocks runs while the late ones are still in flight.
// Arithmetic and summation orders are those of pair_gateup_item.
// ------------------------------------------------------------------------------------------------
constexpr int kWideWarps = 16;
#ifndef EXMOE_WIDE_MAX_PAIRS
#define EXMOE_WIDE_MAX_PAIRS 32
#endif
constexpr int kWideMaxPairs = EXMOE_WIDE_MAX_PAIRS;     // pairs up to which the wide gate/up kernel is taken
#ifndef EXMOE_WIDE_AHEAD
#define EXMOE_WIDE_AHEAD 4
#endif

// one 128-wide block of a unit: gate and up words in registers, activations of the warp's K range in `xr`
__device__ __forceinline__ void wide_block(const uint4 (&wb)[2][2], const uint32_t (&sb)[2], float adj, int b,
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

template <int NB>
__global__ void __launch_bounds__(32 * kWideWarps, 1)
pair_gateup_wide_kernel(GemmArgs a, SmallArgs sa, const __nv_bfloat16* __restrict__ hidden,
                        __nv_bfloat16* __restrict__ act_out, int ks_log2) {
    // grid = (slices of 16 >> ks_log2 panel pairs, selected expert j, token t): pair p = t * k + j
    extern __shared__ __align__(128) unsigned char smem[];
    // Launched as a programmatic dependent of whatever precedes it in the stream (in a decode loop the previous layer
    // call's down kernel, which releases its dependents when it starts): the CTAs are placed and wait here, so the
    // launch latency is off the step; nothing is read or written before the wait.
    grid_dependency_wait();
    grid_launch_dependents();
    if ((blockIdx.x | blockIdx.y | blockIdx.z) == 0) keep_pair_ids(sa);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int p = blockIdx.z * a.top_k + blockIdx.y;
    const int KB = a.H / kGroup, KS = 1 << ks_log2, PP = kWideWarps >> ks_log2;
    const int ks = warp & (KS - 1), pp = warp >> ks_log2;
    unsigned char* xw = smem + (size_t)warp * NB * kGroup * 2;                  // this warp's K range of the hidden row
    float* red = reinterpret_cast<float*>(smem + (size_t)kWideWarps * NB * kGroup * 2);   // [PP][KS][2][16]

    // the hidden row does not depend on the ids: request this warp's K range of it first
    constexpr int XL = (NB * 16 + 31) / 32;                                      // 16-byte chunks per lane
    const unsigned char* xrow = reinterpret_cast<const unsigned char*>(hidden + (size_t)blockIdx.z * a.H) + (size_t)ks * NB * kGroup * 2;
    uint4 xpre[XL];
#pragma unroll
    for (int i = 0; i < XL; ++i) {
        xpre[i] = make_uint4(0, 0, 0, 0);
        if (i * 32 + lane < NB * 16) xpre[i] = ldg_early128(xrow + (size_t)(i * 32 + lane) * 16);
    }
    const int id = sa.ids[p];
    if (id < 0 || id >= sa.E) return;                  // uniform over the CTA; the pair contributes nothing
    const int slot = sa.slot_of ? sa.slot_of[id] : id;
    const int panel = blockIdx.x * PP + pp;
    const uint8_t* base = a.slots + (size_t)slot * a.slot_stride + ((size_t)(2 * panel) * KB + (size_t)ks * NB) * kBlockBytes;
    uint4 wreg[NB][2][2];
    uint32_t sreg[NB][2];
    auto issue_block = [&](int b) {
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const uint8_t* blk = base + ((size_t)m * KB + b) * kBlockBytes;
            wreg[b][m][0] = ldg_stream128(blk + lane * 16);
            wreg[b][m][1] = ldg_stream128(blk + 512 + lane * 16);
            sreg[b][m] = ldg_stream32(blk + kCodeBytes + q * 4);
        }
    };
    constexpr int AHEAD = EXMOE_WIDE_AHEAD < NB ? EXMOE_WIDE_AHEAD : NB;         // blocks requested before the arithmetic starts
#pragma unroll
    for (int b = 0; b < AHEAD; ++b) issue_block(b);
    float adjv[NB];
#pragma unroll
    for (int i = 0; i < XL; ++i) {
        const int ck = i * 32 + lane;
        if (ck < NB * 16) *reinterpret_cast<uint4*>(xw + ck * 16) = xpre[i];
        float sx = sum8_bf16(xpre[i]);
#pragma unroll
        for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
        const float lo = __shfl_sync(0xffffffffu, sx, 0), hi = __shfl_sync(0xffffffffu, sx, 16);
        // __fmul_rn: the product is rounded on its own, as where pair_gateup_item keeps it in shared memory (left to the
        // compiler it would be contracted into the accumulator addition that consumes it: different bits)
        if (2 * i < NB) adjv[2 * i] = __fmul_rn(-136.f, lo);
        if (2 * i + 1 < NB) adjv[2 * i + 1] = __fmul_rn(-136.f, hi);
    }
    __syncwarp();
    float tot[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (b + AHEAD < NB) issue_block(b + AHEAD);
        wide_block(wreg[b], sreg[b], adjv[b], b, xw, lane, tot);
    }
    if (c == 0) {
        float* r = red + (size_t)warp * 32;            // warp = pp * KS + ks
        r[q] = tot[0][0];
        r[q + 8] = tot[0][1];
        r[16 + q] = tot[1][0];
        r[16 + q + 8] = tot[1][1];
    }
    __syncthreads();
    // K ranges added in ascending order, SwiGLU, one rounding to BF16
    if (tid < PP * kPanelRows) {
        const int spp = tid >> 4, r = tid & 15;
        const float* rb = red + ((size_t)spp << ks_log2) * 32;
        float g = rb[r], u = rb[16 + r];
        for (int s2 = 1; s2 < KS; ++s2) {
            g += rb[s2 * 32 + r];
            u += rb[s2 * 32 + 16 + r];
        }
        act_out[(size_t)p * a.I + (size_t)(blockIdx.x * PP + spp) * kPanelRows + r] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * u);
    }
}

// ------------------------------------------------------------------------------------------------
// Bulk-copy variant of the by-token down kernel, used for two or more tokens.  Each expert warp brings its
// panel (one contiguous range of the packed image) into SHARED MEMORY with one cp.async.bulk, completion counted
// in bytes on an mbarrier, instead of into registers: the CTA is light in registers, all of its weight bytes are
// requested in its first instructions (before the dependency on the gate/up kernel), and the MMA loop reads
// them back in lane order.  Measured (OLMoE shape): T=2 19.3 us per step against 22.2 us with the register
// kernel, T=3 27.0 against 31.4; at T=1 the register kernel overlaps the gate/up kernel better (12.9 against
// 13.9 us) and stays.  A bulk-copy gate/up kernel (two-stage ring, one CTA per SM) measured slower at every
// size (T=1: 15.0 us per step) and was dropped.  Arithmetic and summation order are those of
// token_down_kernel (same bits).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void bulk_load_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// after a failed wait: give copies that may still be in flight a bounded time to land before the CTA ends
__device__ __forceinline__ void drain_bar(uint64_t* bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try(bar, parity) && clock64() - t0 < kWaitBudget) {}
}

template <int NBT>
__global__ void __launch_bounds__(256, 1)
token_down_bulk_kernel(GemmArgs a, SmallArgs sa, const __nv_bfloat16* __restrict__ act, const float* __restrict__ topk_w,
                       int bpwg) {
    extern __shared__ __align__(128) unsigned char smem[];
    grid_launch_dependents();                          // the next kernel in the stream may be placed (it waits for this one)
    const int K = a.I, KB = K / kGroup, k = a.top_k;                     // k <= 8: one warp per selected expert
    const uint32_t panel_bytes = (uint32_t)KB * kBlockBytes;
    const int x_stride = K * 2 + 64;
    unsigned char* wst = smem;                                           // [k][panel_bytes]
    unsigned char* xs = smem + (size_t)k * panel_bytes;                  // [k][x_stride]
    float* ys = reinterpret_cast<float*>(xs + (size_t)k * x_stride);     // [k][16]
    int* s_valid = reinterpret_cast<int*>(ys + k * 16);                  // [k]
    float* adj = reinterpret_cast<float*>(s_valid + 8);                  // [KB][k]
    uint64_t* bar = reinterpret_cast<uint64_t*>(adj + (((size_t)KB * k + 3) & ~(size_t)3));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar + 1);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int t = blockIdx.y, panel = blockIdx.x;                        // grid = (16-row panels of the output, tokens)
    if (tid == 0) {
        mbar_init(bar, k);                                               // one arrival per expert warp
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int j = warp;
    const int pair = t * k + j;
    int id = -1;
    if (j < k) id = sa.ids[pair];
    const bool valid = (j < k) && id >= 0 && id < sa.E;
    const float rw = valid ? ldg_early_f32(topk_w + pair) : 0.f;
    if (j < k && lane == 0) {                                            // the expert's panel: one contiguous range
        if (valid) {
            const int slot = sa.slot_of ? sa.slot_of[id] : id;
            const uint8_t* src = a.slots + (size_t)slot * a.slot_stride + matrix_bytes(2 * a.I, a.H) + (size_t)panel * panel_bytes;
            mbar_expect_tx(bar, panel_bytes);
            bulk_load_g2s(wst + (size_t)j * panel_bytes, src, panel_bytes, bar);
        } else {
            mbar_arrive(bar);
        }
    }
    grid_dependency_wait();                                              // the gate/up kernel's activations are complete and visible
    {
        // four 16-byte chunks per thread in flight at once (one L2 round trip per batch), then the block sums
        const int chunks_per_row = K / 8, total = k * chunks_per_row;
        const int cpr_shift = (chunks_per_row & (chunks_per_row - 1)) ? -1 : __ffs(chunks_per_row) - 1;
        const uint4* src = reinterpret_cast<const uint4*>(act + (size_t)t * k * K);         // the token's k rows are contiguous
        for (int base0 = warp * 32; base0 < total; base0 += 4 * 256) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base0 + u * 256 + lane;
                v[u] = make_uint4(0, 0, 0, 0);
                if (idx < total) v[u] = __ldcg(src + idx);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base0 + u * 256 + lane;
                int n, ck;
                if (cpr_shift >= 0) {                  // the usual case: no division between the wait and the MMAs
                    n = idx >> cpr_shift;
                    ck = idx & (chunks_per_row - 1);
                } else {
                    n = idx / chunks_per_row;
                    ck = idx - n * chunks_per_row;
                }
                if (idx < total) *reinterpret_cast<uint4*>(xs + (size_t)n * x_stride + ck * 16) = v[u];
                float sx = sum8_bf16(v[u]);
#pragma unroll
                for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
                if (idx < total && (ck & 15) == 0) adj[(ck >> 4) * k + n] = -136.f * sx;
            }
        }
    }
    __syncthreads();
    const bool ok = mbar_wait(bar, 0, abort_flag, sa.status);
    float result[2] = {0.f, 0.f}, total2[2] = {0.f, 0.f};
    if (valid) {
        const unsigned char* mine = wst + (size_t)j * panel_bytes;
        for (int b0 = 0; b0 < KB; b0 += NBT) {
#pragma unroll
            for (int b = 0; b < NBT; ++b) {
                const unsigned char* blk = mine + (size_t)(b0 + b) * kBlockBytes;
                const uint4 w0 = *reinterpret_cast<const uint4*>(blk + lane * 16);
                const uint4 w1 = *reinterpret_cast<const uint4*>(blk + 512 + lane * 16);
                const uint32_t sv = *reinterpret_cast<const uint32_t*>(blk + kCodeBytes + q * 4);
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int set = 0; set < 2; ++set) {
                        const int k0 = (b0 + b) * kGroup + 64 * h + 32 * set + 8 * c;
                        uint4 xb = make_uint4(0, 0, 0, 0);
                        if (q == 0) xb = *reinterpret_cast<const uint4*>(xs + (size_t)j * x_stride + k0 * 2);
                        const uint4& wh = h ? w1 : w0;
                        const uint32_t wq = set ? wh.z : wh.x;
                        const uint32_t wq8 = set ? wh.w : wh.y;
                        mma_m16n8k16(acc, code_pair(wq, 0), code_pair(wq8, 0), code_pair(wq, 4), code_pair(wq8, 4), xb.x, xb.y);
                        mma_m16n8k16(acc, code_pair(wq, 8), code_pair(wq8, 8), code_pair(wq, 12), code_pair(wq8, 12), xb.z, xb.w);
                    }
                const __half2 sc = *reinterpret_cast<const __half2*>(&sv);
                const float cr = adj[(b0 + b) * k + j];
                total2[0] = fmaf(__low2float(sc), acc[0] + cr, total2[0]);
                total2[1] = fmaf(__high2float(sc), acc[2] + cr, total2[1]);
                if ((b0 + b + 1) % bpwg == 0) {                          // end of one K-split range of the grouped kernel
                    const bool first = (b0 + b + 1 == bpwg);
                    result[0] = first ? total2[0] : result[0] + total2[0];
                    result[1] = first ? total2[1] : result[1] + total2[1];
                    total2[0] = total2[1] = 0.f;
                }
            }
        }
    }
    if (j < k) {
        if (lane == 0) s_valid[j] = valid ? 1 : 0;
        if (c == 0) {
            ys[j * 16 + q] = rw * result[0];
            ys[j * 16 + q + 8] = rw * result[1];
        }
    }
    __syncthreads();
    if (tid < 16 && ok) {
        float sum = 0.f;
        for (int jj = 0; jj < k; ++jj)
            if (s_valid[jj]) sum += ys[jj * 16 + tid];
        sa.out[(size_t)t * a.H + panel * kPanelRows + tid] = __float2bfloat16_rn(sum);
    }
    if (!ok && tid == 0) drain_bar(bar, 0);
}

// launch with programmatic stream serialisation: the grid may be placed while its predecessor in the stream still runs
// (once that has released its dependents); the kernel itself waits (griddepcontrol.wait) before it touches memory
template <typename Kern, typename... Args>
static void launch_pdl(Kern kern, dim3 grid, int block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t lc{};
    lc.gridDim = grid;
    lc.blockDim = dim3(block);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
#ifdef EXMOE_DISABLE_PDL
    lc.numAttrs = 0;
#endif
    cudaLaunchKernelEx(&lc, kern, args...);
}

template <int NB>
void launch_pair_gateup(const GemmArgs& a, const SmallArgs& sa, const __nv_bfloat16* hidden, __nv_bfloat16* act, int KS,
                        cudaStream_t st) {
    auto kern = pair_gateup_kernel<NB>;
    const int PP = 8 / KS, tiles = a.I / (kPanelRows * PP);
    const size_t smem = (size_t)a.H * 2 + 64 + (size_t)(KS - 1) * PP * 2 * 128 * 4 + (size_t)(a.H / kGroup) * 4;
    static SmemOnce smem_once;
    allow_smem(kern, 100 * 1024, smem_once);
    int ks_log2 = 0;
    while ((1 << ks_log2) < KS) ++ks_log2;
    launch_pdl(kern, dim3(tiles, a.top_k, sa.n_pairs / a.top_k), 256, smem, st, a, sa, hidden, act, ks_log2);
    count_launch();
}

// false when the shape does not fit the wide kernel (the caller then takes pair_gateup_kernel)
template <int NB>
bool launch_pair_gateup_wide(const GemmArgs& a, const SmallArgs& sa, const __nv_bfloat16* hidden, __nv_bfloat16* act, int KS,
                             cudaStream_t st) {
#ifdef EXMOE_NO_WIDE_GATEUP
    return false;
#endif
    int ks_log2 = 0;
    while ((1 << ks_log2) < KS) ++ks_log2;
    const int PP = kWideWarps >> ks_log2;
    if ((1 << ks_log2) != KS || PP < 1 || a.I % (kPanelRows * PP)) return false;
    auto kern = pair_gateup_wide_kernel<NB>;
    const size_t smem = (size_t)kWideWarps * NB * kGroup * 2 + (size_t)kWideWarps * 32 * 4;
    static SmemOnce smem_once;
    allow_smem(kern, 100 * 1024, smem_once);
    launch_pdl(kern, dim3(a.I / (kPanelRows * PP), a.top_k, sa.n_pairs / a.top_k), 32 * kWideWarps, smem, st, a, sa, hidden, act,
               ks_log2);
    count_launch();
    return true;
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

template <int NB, int NCH, bool GATEUP, int MODE>
void launch_cfg(const GemmArgs& a, const SmallArgs& sa, const __nv_bfloat16* x, __nv_bfloat16* act, const float* w,
                float* y, const DecodeCfg& cfg, int max_groups, cudaStream_t st) {
    constexpr int NM = GATEUP ? 2 : 1;
    const int K = GATEUP ? a.H : a.I, NR = GATEUP ? a.I : a.H;
    const int PP = 8 / cfg.KS;
    const int tiles = NR / (kPanelRows * PP);
    size_t smem = (size_t)8 * NCH * (K * 2 + 64) + (size_t)(cfg.KS - 1) * PP * NM * NCH * 128 * 4 +
                  (size_t)(K / kGroup) * 8 * NCH * 4;
    constexpr bool SMALL = (MODE == MODE_SMALL);
    if (SMALL) smem += (size_t)(3 * a.num_slots + 1 + 2 * sa.n_pairs) * 4;
    auto kern = decode_gemm_kernel<NB, NCH, GATEUP, MODE>;
    static SmemOnce smem_once;                      // per instantiation
    allow_smem(kern, 200 * 1024, smem_once);
    long long items = (long long)max_groups * tiles;
    const int grid = (int)(items < 148 * 8 ? (items < 1 ? 1 : items) : 148 * 8);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(256);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (SMALL && !GATEUP) ? 1 : 0;           // only the down kernel overlaps its predecessor
#ifdef EXMOE_DISABLE_PDL
    lc.numAttrs = 0;
#endif
    cudaLaunchKernelEx(&lc, kern, a, sa, x, act, w, y, cfg.KS, cfg.bpw);
    count_launch();
}

template <bool GATEUP, int MODE>
void launch_decode(const GemmArgs& a, const SmallArgs& sa, const __nv_bfloat16* x, __nv_bfloat16* act, const float* w,
                   float* y, int max_rows, int max_groups, cudaStream_t st) {
    const int K = GATEUP ? a.H : a.I, NR = GATEUP ? a.I : a.H;
    const DecodeCfg cfg = pick_cfg(K, NR);
    // rows per pass: one 8-row chunk covers decode; more chunks amortise the dequantisation
    int nch = max_rows <= 8 ? 1 : (max_rows <= 16 ? 2 : 4);
    while (nch > 1 && (size_t)8 * nch * (K * 2 + 64) > 150 * 1024) nch >>= 1;
#define EXMOE_DISPATCH(NBv)                                                                                   \
    if (nch == 1) launch_cfg<NBv, 1, GATEUP, MODE>(a, sa, x, act, w, y, cfg, max_groups, st);                 \
    else if (MODE == MODE_PAIR) return;                                                                       \
    else if (nch == 2) launch_cfg<NBv, 2, GATEUP, MODE>(a, sa, x, act, w, y, cfg, max_groups, st);            \
    else launch_cfg<NBv, 4, GATEUP, MODE>(a, sa, x, act, w, y, cfg, max_groups, st);
    if (cfg.NB == 4) { EXMOE_DISPATCH(4) }
    else if (cfg.NB == 2) { EXMOE_DISPATCH(2) }
    else { EXMOE_DISPATCH(1) }
#undef EXMOE_DISPATCH
}

// out[t] = bf16( sum_{j=0..k-1} Y[t*k + j] ), binary32, fixed order; pairs with an invalid id add nothing
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ y, const int32_t* __restrict__ ids, int E, int T, int k, int H,
               __nv_bfloat16* __restrict__ out) {
    grid_launch_dependents();                          // the next kernel in the stream may be placed (it waits for this one)
    const int per_row = H / 4;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    grid_dependency_wait();                            // launched as a programmatic dependent of the down kernel
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

void launch_combine(const float* y, const int32_t* ids, int E, int T, int k, int H, __nv_bfloat16* out,
                    cudaStream_t st) {
    const long long n = (long long)T * (H / 4);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)((n + 255) / 256));
    lc.blockDim = dim3(256);
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
#ifdef EXMOE_DISABLE_PDL
    lc.numAttrs = 0;
#endif
    cudaLaunchKernelEx(&lc, combine_kernel, y, ids, E, T, k, H, out);
    count_launch();
}


template <int NBT>
void launch_token_down(const GemmArgs& a, const SmallArgs& sa, const __nv_bfloat16* act, const float* w, int T,
                       int bpwg, cudaStream_t st) {
    auto kern = token_down_kernel<NBT>;
    const size_t smem = (size_t)a.top_k * (a.I * 2 + 64) + (size_t)a.top_k * 17 * 4 + (size_t)(a.I / kGroup) * a.top_k * 4;
    static SmemOnce smem_once;
    allow_smem(kern, 200 * 1024, smem_once);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(T * (a.H / kPanelRows));
    lc.blockDim = dim3(256);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
#ifdef EXMOE_DISABLE_PDL
    lc.numAttrs = 0;
#endif
    cudaLaunchKernelEx(&lc, kern, a, sa, act, w, bpwg);
    count_launch();
}

// false when the shape does not fit the kernel's shared-memory budget (the caller then takes the register variant)
template <int NBT>
bool launch_token_down_bulk(const GemmArgs& a, const SmallArgs& sa, const __nv_bfloat16* act, const float* w, int T, int bpwg,
                            cudaStream_t st) {
    const int K = a.I, KB = K / kGroup, k = a.top_k;
    if (k > 8) return false;
    const size_t smem = (size_t)k * KB * kBlockBytes + (size_t)k * (K * 2 + 64) + (size_t)k * 16 * 4 + 32 +
                        (((size_t)KB * k + 3) & ~(size_t)3) * 4 + 64;
    if (smem > 100 * 1024) return false;
    auto kern = token_down_bulk_kernel<NBT>;
    static SmemOnce smem_once;
    allow_smem(kern, 100 * 1024, smem_once);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(a.H / kPanelRows, T);
    lc.blockDim = dim3(256);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
#ifdef EXMOE_DISABLE_PDL
    lc.numAttrs = 0;
#endif
    cudaLaunchKernelEx(&lc, kern, a, sa, act, w, bpwg);
    count_launch();
    return true;
}

// Shared memory the per-pair kernels ask for (launch_pair_gateup, launch_token_down): false when either exceeds its
// opt-in limit, so that callers can refuse or take another path BEFORE anything is queued.
bool pair_path_fits(int H, int I, int top_k) {
    const DecodeCfg cfg = pick_cfg(H, I);
    const int PP = 8 / cfg.KS;
    const size_t gu = (size_t)H * 2 + 64 + (size_t)(cfg.KS - 1) * PP * 2 * 128 * 4 + (size_t)(H / kGroup) * 4;
    const size_t dn = (size_t)top_k * (I * 2 + 64) + (size_t)top_k * 17 * 4 + (size_t)(I / kGroup) * top_k * 4;
    return gu <= 100 * 1024 && dn <= 200 * 1024 && (cfg.bpw == 1 || cfg.bpw == 2 || cfg.bpw == 4);
}
// ... and the in-CTA-grouping kernels with one 8-row chunk per pass (their smallest footprint)
bool small_path_fits(int H, int I, int num_slots, int n_pairs) {
    for (int g = 0; g < 2; ++g) {
        const int K = g ? I : H, NR = g ? H : I;
        const DecodeCfg cfg = pick_cfg(K, NR);
        const int PP = 8 / cfg.KS, NM = g ? 1 : 2;
        const size_t smem = (size_t)8 * (K * 2 + 64) + (size_t)(cfg.KS - 1) * PP * NM * 128 * 4 + (size_t)(K / kGroup) * 8 * 4 +
                            (size_t)(3 * num_slots + 1 + 2 * n_pairs) * 4;
        if (smem > 200 * 1024) return false;
    }
    return true;
}

// One wave of the SMALL path: gate/up kernel, then the down kernel with the fused combine.
void launch_small_wave(const GemmArgs& a, const SmallWave& w, cudaStream_t st, bool gateup, bool down) {
    SmallArgs sa{};
    sa.ids = w.ids;
    sa.wave_of = w.wave_of;
    sa.slot_of = w.slot_of;
    sa.n_pairs = w.n_pairs;
    sa.E = w.E;
    sa.wave = w.wave;
    sa.pub_counts = w.plan.counts;
    sa.pub_offsets = w.plan.offsets;
    sa.pub_perm = w.plan.perm;
    sa.header = w.plan.header;
    sa.status = w.status;
    sa.arrive = w.arrive;
    sa.out = w.out;
    sa.saved_ids = w.saved_ids;
    if (w.pairwise) {                                   // T*k <= 32, one wave: no grouping, by-token down + combine
        if (gateup) {
            const DecodeCfg cfg = pick_cfg(a.H, a.I);
            // one token: the wide kernel (one 16-warp CTA per SM, every warp its own load/convert pipeline)
            const bool wide = w.n_pairs <= kWideMaxPairs;
            if (cfg.bpw == 4 && wide && launch_pair_gateup_wide<4>(a, sa, w.hidden, w.act, cfg.KS, st)) {}
            else if (cfg.bpw == 2 && wide && launch_pair_gateup_wide<2>(a, sa, w.hidden, w.act, cfg.KS, st)) {}
            else if (cfg.bpw == 1 && wide && launch_pair_gateup_wide<1>(a, sa, w.hidden, w.act, cfg.KS, st)) {}
            else if (cfg.bpw == 4) launch_pair_gateup<4>(a, sa, w.hidden, w.act, cfg.KS, st);
            else if (cfg.bpw == 2) launch_pair_gateup<2>(a, sa, w.hidden, w.act, cfg.KS, st);
            else if (cfg.bpw == 1) launch_pair_gateup<1>(a, sa, w.hidden, w.act, cfg.KS, st);
            else launch_decode<true, MODE_PAIR>(a, sa, w.hidden, w.act, nullptr, nullptr, 1, w.n_pairs, st);
        }
        if (down) {
            const int KB = a.I / kGroup;
            const int bpwg = pick_cfg(a.I, a.H).bpw;    // the grouped kernel's K-split range, replayed for rounding
            const int T = w.n_pairs / a.top_k;
            bool done = false;
#ifndef EXMOE_NO_BULK_DECODE
            if (T >= 2) {                               // one token: the register kernel overlaps the gate/up kernel better
                if (KB % 8 == 0) done = launch_token_down_bulk<8>(a, sa, w.act, w.topk_w, T, bpwg, st);
                else if (KB % 4 == 0) done = launch_token_down_bulk<4>(a, sa, w.act, w.topk_w, T, bpwg, st);
                else if (KB % 2 == 0) done = launch_token_down_bulk<2>(a, sa, w.act, w.topk_w, T, bpwg, st);
                else done = launch_token_down_bulk<1>(a, sa, w.act, w.topk_w, T, bpwg, st);
            }
#endif
            if (done) {}
            else if (KB % 8 == 0) launch_token_down<8>(a, sa, w.act, w.topk_w, T, bpwg, st);
            else if (KB % 4 == 0) launch_token_down<4>(a, sa, w.act, w.topk_w, T, bpwg, st);
            else if (KB % 2 == 0) launch_token_down<2>(a, sa, w.act, w.topk_w, T, bpwg, st);
            else launch_token_down<1>(a, sa, w.act, w.topk_w, T, bpwg, st);
        }
        return;
    }
    if (gateup) launch_decode<true, MODE_SMALL>(a, sa, w.hidden, w.act, nullptr, nullptr, w.max_rows, w.max_groups, st);
    if (down) launch_decode<false, MODE_SMALL>(a, sa, w.act, nullptr, w.topk_w, w.y, w.max_rows, w.max_groups, st);
}

// ------------------------------------------------------------------------------------------------
// Allocation-free tiny-batch forward (exmoe_moe_forward_static).
//
// The pairwise kernels need scratch: the BF16 SwiGLU activations handed from the gate/up kernel to
// the down kernel, plus a status word and the kept ids.  exmoe_moe_forward takes that scratch from
// the workspace the caller allocated for the cache.  This entry point serves callers that can hand
// over no scratch at all: it lives in the fixed array below, which every GPU that loads this
// library holds until the process exits.
// ------------------------------------------------------------------------------------------------
constexpr int kStaticMaxPairs = kPairMaxPairs;           // T * top_k <= 32
constexpr int kStaticMaxDff = 4096;                      // d_ff <= 4096
constexpr size_t kStaticCtrlBytes = 256;                 // [32,36) sticky status word, [64,192) kept ids
constexpr size_t kStaticScratchBytes = kStaticCtrlBytes + (size_t)kStaticMaxPairs * kStaticMaxDff * 2;   // 262,400 B

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

}  // namespace exmoe

#include <mutex>

// Device address of the scratch on the current device (set-up once per device, see exmoe_moe_forward_static).
static unsigned char* static_scratch_ptr() {
    static std::mutex mu;
    static unsigned char* dev_ptr[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!dev_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, exmoe::g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return nullptr;
        }
        dev_ptr[dev] = static_cast<unsigned char*>(p);
    }
    return dev_ptr[dev];
}

extern "C" int exmoe_moe_forward_static_status(void) {
    unsigned char* scratch = static_scratch_ptr();
    if (!scratch) return EXMOE_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, scratch + 32, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return EXMOE_ERR_CUDA;
    if (v && cudaMemset(scratch + 32, 0, 4) != cudaSuccess) return EXMOE_ERR_CUDA;
    return v;
}

extern "C" int exmoe_moe_forward_static(const exmoe_shape* shape, const void* experts_dev, const void* hidden_bf16,
                                        const int32_t* topk_ids, const float* topk_weights, int T, void* out_bf16,
                                        void* stream) {
    using namespace exmoe;
    if (!shape || T < 0) return EXMOE_ERR_ARG;
    if (shape->group_size != kGroup || shape->d_model <= 0 || shape->d_ff <= 0 || shape->d_model % kGroup ||
        shape->d_ff % kGroup || shape->num_experts <= 0 || shape->top_k <= 0 || shape->top_k > shape->num_experts)
        return EXMOE_ERR_SHAPE;
    // the fixed scratch bounds the problem: reject anything larger instead of overrunning it
    if ((long long)T * shape->top_k > kStaticMaxPairs || shape->d_ff > kStaticMaxDff) return EXMOE_ERR_SHAPE;
    // ... and so does the shared memory of the two kernels (e.g. top_k = 32 with d_ff = 4096 would ask for 264 KB)
    if (!pair_path_fits(shape->d_model, shape->d_ff, shape->top_k)) return EXMOE_ERR_SHAPE;
    if (T == 0) return EXMOE_OK;
    if (!experts_dev || !hidden_bf16 || !topk_ids || !topk_weights || !out_bf16) return EXMOE_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(experts_dev) | reinterpret_cast<uintptr_t>(hidden_bf16) |
         reinterpret_cast<uintptr_t>(out_bf16)) & 15)
        return EXMOE_ERR_ARG;

    // Set-up, once per device, with that device current: in host code `g_static_scratch` is only a
    // stand-in for the symbol, not a device address; the address a kernel may use comes from
    // cudaGetSymbolAddress (static_scratch_ptr).
    unsigned char* scratch = static_scratch_ptr();
    if (!scratch) return EXMOE_ERR_CUDA;

    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps the previous call's contents: the kept ids must start clean; the status word at [32, 36) is
    // sticky on purpose (exmoe_moe_forward_static_status reads and clears it)
    if (cudaMemsetAsync(scratch + 64, 0, kStaticCtrlBytes - 64, st) != cudaSuccess) return EXMOE_ERR_CUDA;

    GemmArgs a{};
    a.slots = static_cast<const uint8_t*>(experts_dev);
    a.slot_stride = matrix_bytes(2 * shape->d_ff, shape->d_model) + matrix_bytes(shape->d_model, shape->d_ff);
    a.num_slots = shape->num_experts;
    a.top_k = shape->top_k;
    a.H = shape->d_model;
    a.I = shape->d_ff;
    SmallWave w{};
    w.ids = topk_ids;
    w.n_pairs = T * shape->top_k;
    w.E = shape->num_experts;
    w.wave = 0;
    w.status = reinterpret_cast<int*>(scratch + 32);
    w.saved_ids = reinterpret_cast<int32_t*>(scratch + 64);
    w.hidden = static_cast<const __nv_bfloat16*>(hidden_bf16);
    w.act = reinterpret_cast<__nv_bfloat16*>(scratch + kStaticCtrlBytes);
    w.topk_w = topk_weights;
    w.out = static_cast<__nv_bfloat16*>(out_bf16);
    w.max_rows = T;
    w.max_groups = w.n_pairs;
    w.pairwise = true;
    launch_small_wave(a, w, st, true, true);
    return cudaGetLastError() == cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}
