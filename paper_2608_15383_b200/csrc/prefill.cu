// Large-M grouped W4A16 GEMMs on the 5th-generation tensor cores (prefill; the two grouped expert
// GEMMs per wave of Section 3.4 / Eq. 2 when every expert has many rows).
//
// Swap-AB: the WEIGHTS are the UMMA A operand (M = 128 rows = 8 consecutive 16-row panels of the
// packed matrix), the TOKENS are the B operand (N <= 256 grouped rows), the accumulator D[128 x N]
// lives in TMEM (fp32, lane = weight row, column = token).  For gate/up the 8 panels are
// gate p, up p, gate p+1, ... so one accumulator holds 64 intermediates' gate rows and up rows
// 16 lanes apart: SwiGLU is one shuffle away in the epilogue.
//
// A persistent CTA (one per SM, 28 warps) is specialised by warp:
//   warp 0        allocates TMEM, then ONE thread issues tcgen05.mma (4 x K16 per 64-wide ring stage) and
//                 tcgen05.commit to the stage-empty / accumulator-full mbarriers, from an unrolled ring
//                 (see the note at the issue loop: what bounds this kernel is what that thread does between MMAs).
//   warps 4-7,    epilogue (two groups, even / odd 32-column chunks): tcgen05.ld the accumulator (warp w
//   16-19         reads TMEM lanes 32(w%4)..), SwiGLU -> BF16 activations, or routing weight -> fp32
//                 pair buffer; two accumulators (2 x 256 columns) let the epilogue of tile i overlap
//                 the MMAs of tile i+1.
//   warp 1        B producer: one thread issues one TMA tile load (cp.async.bulk.tensor.2d, 128-byte
//                 swizzle, the tile's rows x 64 columns) per stage from the grouped activation matrix;
//                 completion is counted in bytes on the stage's full barrier.  No multicast.
//   warps 8-15,   A producers, one 16-row panel and one 64-wide k-half (= every second stage) each: stream
//   20-27         packed int4 (128-bit loads, two blocks ahead in registers), dequantise to BF16 (shift/lop3 ->
//                 128+u, subtract 136, multiply by the exactly split group scale: one rounding) and store the
//                 canonical no-swizzle K-major core-matrix layout (k-chunk stride padded to 160 bytes:
//                 conflict-free stores).
// Producers -> MMA through full[stage] mbarriers (generic-proxy writes are fenced with
// fence.proxy.async before the arrive), MMA -> producers through tcgen05.commit on empty[stage].
// The gate/up GEMM reads its tokens from a grouped copy of the hidden states (rows in plan order),
// written once per call by gather_rows_kernel, so that both GEMMs load B with plain tiled TMA.
// Every wait is bounded: on expiry the CTA raises EXMOE_ERR_TIMEOUT, all roles drain, TMEM is freed.
//
// Measured alone on one SM (one CTA, operands in place): an MMA of this shape takes N / 2 cycles issued back to
// back, from shared-memory A as from tensor-memory A, and its issue blocks while the pipe is busy.  Two variants
// of this kernel were built, are parity-green and are in the history, not in the tree: the dequantised weights
// written to TENSOR MEMORY (tcgen05.st.16x256b hands every lane the cells of its mma-fragment-ordered codes up to
// a K permutation inside every 64, which the token matrices were stored in as well) with A taken from there, and
// CTA PAIRS (cta_group::2: M = 256, each CTA dequantises its 128 rows and fetches half of the token tile, one
// commit multicast to both).  On config 4 they measured 338 and 344 us per step against 323 us for this one:
// tensor memory leaves room for 192-row tiles only (more tiles, more conversion work), the pair halves neither
// the conversion work nor, it turned out, the time.
#include <cuda.h>

#include "common.cuh"
#include "mbar.cuh"
#ifdef EXMOE_PREFILL_PROF
#include <cstdio>
#endif

namespace exmoe {

namespace {

constexpr int BM = 128;            // weight rows per tile
constexpr int BN = 256;            // max grouped rows (tokens) per tile of the large-N kernel shape
constexpr int BN_SMALL = 64;       // ... and of the small-N shape (a few dozen rows per expert: eight stages fit)
constexpr int BK = 128;            // one packed block / one scale group
constexpr int BKS = 64;            // K per ring stage = half a packed block (the half one dequantisation warp converts)
// A (dequantised weights): no swizzle; core matrix = 8 rows x 16 B; k-chunks 160 B apart (128 + 32 pad, so that
// the 8 lanes of a quarter warp, 2 rows x 4 k-chunks, hit 8 different 16-byte bank groups), row groups 1280 B apart
constexpr int A_LBO = 160;
constexpr int A_SBO = (BKS / 8) * A_LBO;
constexpr int A_STAGE_BYTES = 16 * A_SBO;      // 20 KB
// B (tokens): TMA 128-byte swizzle; 64 columns x up to 256 rows of 128 B; 8-row atoms of 1024 B
constexpr int B_SBO = 1024;
constexpr int N_MAPS = 16;         // tensor maps per operand: boxes of 16, 32, ..., 256 rows
constexpr int NUM_THREADS = 896;   // 28 warps: MMA, TMA, 2 idle, 4 + 4 epilogue, 8 + 8 dequant

struct Tile { int key, n0, nrows, pad; };

#ifdef EXMOE_PREFILL_PROF
#define PROF_DECL long long prof_t0 = clock64(), prof_wait = 0
#define PROF_WAIT_BEGIN long long prof_w0 = clock64()
#define PROF_WAIT_END prof_wait += clock64() - prof_w0
#define PROF_REPORT(name) if (blockIdx.x == 7 && lane == 0) printf("%s warp %d: total %lld wait %lld\n", name, warp, clock64() - prof_t0, prof_wait)
#else
#define PROF_DECL
#define PROF_WAIT_BEGIN
#define PROF_WAIT_END
#define PROF_REPORT(name)
#endif

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared-memory matrix descriptors, K-major, version 1 (sm_100)
__device__ __forceinline__ uint64_t make_desc_a(uint32_t saddr) {            // no swizzle
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)((A_LBO >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((A_SBO >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
__device__ __forceinline__ uint64_t make_desc_b(uint32_t saddr) {            // 128-byte swizzle
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)1 << 16;                                                  // leading offset unused with swizzle
    d |= (uint64_t)((B_SBO >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
// instruction descriptor: D fp32, A/B BF16, both K-major, M = 128, N = n
__device__ __forceinline__ uint32_t make_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
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

// The FP16 group scale s is split exactly into two BF16 numbers, s = hi + lo (hi = bf16(s), lo = s - hi has at most
// four significant bits).  For a code q in [-8, 7]: q*lo is exact in BF16 and fma(q, hi, q*lo) rounds the exact
// product q*s once, so the staged weight is the correctly rounded BF16 of the dequantised value s*q.
struct ScaleSplit { __nv_bfloat162 hi, lo; };
__device__ __forceinline__ ScaleSplit split_scale(float s) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(s);
    const __nv_bfloat16 lo = __float2bfloat16_rn(s - __bfloat162float(hi));
    return ScaleSplit{__nv_bfloat162(hi, hi), __nv_bfloat162(lo, lo)};
}
// eight codes of one word -> eight BF16 weights bf16(q * s), K order, as one 16-byte value
__device__ __forceinline__ uint4 dequant_word(uint32_t w, const ScaleSplit& sc) {
    uint32_t bias = 0x43084308u;                                   // BF16 136 twice
    const __nv_bfloat162 b2 = *reinterpret_cast<__nv_bfloat162*>(&bias);
    uint32_t out[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        uint32_t v;
        asm("lop3.b32 %0, %1, 0x000f000f, 0x43004300, 0xea;" : "=r"(v) : "r"(w >> (4 * s)));   // (128+u, 128+u')
        const __nv_bfloat162 q2 = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&v), b2);         // exact small integers
        const __nv_bfloat162 r2 = __hfma2(q2, sc.hi, __hmul2(q2, sc.lo));                       // one rounding of q*s
        out[s] = *reinterpret_cast<const uint32_t*>(&r2);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}

struct PrefillArgs {
    const uint8_t* slots;
    size_t slot_stride;
    const int32_t* perm;
    const Tile* tiles;         // n-tiles of this wave
    const int32_t* n_tiles;    // device scalar
    int num_slots, top_k, H, I;
    int* status;
};

// What an epilogue warp can fetch before the tile's accumulator is complete: the tile's first grouped row and, for the
// down GEMM, the (pair, routing weight) of each of its columns (two dependent global loads per 32-column chunk, which
// cost more than the chunk's stores when they were issued after the wait).
template <int CHUNKS>
struct EpiloguePre {
    int row0;
    int pair[CHUNKS];
    float w[CHUNKS];
};
template <bool GATEUP, int CHUNKS>
__device__ __forceinline__ EpiloguePre<CHUNKS> epilogue_prefetch(const PrefillArgs& a, const Tile& tl, int first, int lane,
                                                                 const int32_t* __restrict__ offsets,
                                                                 const float* __restrict__ topk_w) {
    EpiloguePre<CHUNKS> p;
    p.row0 = offsets[tl.key] + tl.n0;
#pragma unroll
    for (int i = 0; i < CHUNKS; ++i) {
        p.pair[i] = 0;
        p.w[i] = 0.f;
        const int c = first + 64 * i + lane;
        if (!GATEUP && c < tl.nrows) {
            p.pair[i] = a.perm[p.row0 + c];
            p.w[i] = topk_w[p.pair[i]];
        }
    }
    return p;
}
// Epilogue of one tile by one warp: TMEM lanes 32e .. 32e+31 of the accumulator at `tmem_acc`, the 32-column chunks
// c0 = first, first + 64, ...  Gate/up: SwiGLU -> BF16 activations; down: routing weight -> fp32 pair buffer.
template <bool GATEUP, int CHUNKS>
__device__ __forceinline__ void epilogue_tile(const PrefillArgs& a, const Tile& tl, int mt, int e, int first, int lane,
                                              uint32_t tmem_acc, const EpiloguePre<CHUNKS>& pre,
                                              __nv_bfloat16* __restrict__ act_out, float* __restrict__ y_out) {
    const int row0 = pre.row0;
    const uint32_t taddr = tmem_acc + ((uint32_t)(32 * e) << 16);
#pragma unroll
    for (int i = 0; i < CHUNKS; ++i) {
        const int c0 = first + 64 * i;
        if (c0 >= tl.nrows) break;
        uint32_t v[32];
        tc_ld32(taddr + c0, v);
        tc_wait_ld();
        if (GATEUP) {
            // lanes 0-15: gate rows, lanes 16-31: up rows of the same 16 intermediates
            const int interm = (mt * 4 + e) * 16 + (lane & 15);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const uint32_t send = (lane < 16) ? v[j + 16] : v[j];
                const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 16);
                const int col = (lane < 16) ? j : j + 16;
                const float g = __uint_as_float((lane < 16) ? v[j] : recv);
                const float u = __uint_as_float((lane < 16) ? recv : v[j + 16]);
                const int n = c0 + col;
                if (n < tl.nrows)
                    act_out[(size_t)(row0 + n) * a.I + interm] = __float2bfloat16_rn(__fdividef(g, 1.f + __expf(-g)) * u);
            }
        } else {
            const int h = mt * BM + 32 * e + lane;
#pragma unroll
            for (int j = 0; j < 32; ++j) {                 // lane j holds pair and weight of column c0 + j
                const int pair = __shfl_sync(0xffffffffu, pre.pair[i], j);
                const float wj = __shfl_sync(0xffffffffu, pre.w[i], j);
                if (c0 + j < tl.nrows) y_out[(size_t)pair * a.H + h] = wj * __uint_as_float(v[j]);
            }
        }
    }
}

// BN_T = token rows per tile (256 or 64), STAGES = ring depth.  One ring stage holds 64 of K: half a packed block
// of the weights (the half one dequantisation warp converts) and a [rows x 64] box of tokens.  The round trip of one
// stage (MMAs complete -> commit -> token box fetched from L2, weights converted -> MMA issuer wakes) is 2000-3000
// cycles, far more than the stage's MMAs take, so the ring depth sets the rate: 64-wide stages give the large shape
// four of them and the small shape eight in the same shared memory.  The token box holds exactly the tile's rows
// (rounded up to 16): `maps` is a family of tensor maps over the same matrix with boxes of 16, 32, ..., 256 rows.
template <bool GATEUP, int BN_T, int STAGES>
__global__ void __launch_bounds__(NUM_THREADS, 1)
prefill_gemm_kernel(PrefillArgs a, const CUtensorMap* __restrict__ maps, __nv_bfloat16* __restrict__ act_out,
                    const float* __restrict__ topk_w, const int32_t* __restrict__ offsets, float* __restrict__ y_out) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzled tiles need 1 KB alignment
    constexpr int B_STAGE_BYTES = BN_T * 128;                     // BN_T rows x 64 columns
    unsigned char* sB = smem;                                     // [STAGES][B_STAGE_BYTES]
    unsigned char* sA = smem + STAGES * B_STAGE_BYTES;            // [STAGES][20 KB]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sA + STAGES * A_STAGE_BYTES);
    uint64_t* full = bars;                          // [STAGES]  producers -> MMA
    uint64_t* empty = bars + STAGES;                // [STAGES]  MMA -> producers (tcgen05.commit)
    uint64_t* acc_full = bars + 2 * STAGES;         // [2]       MMA -> epilogue
    uint64_t* acc_empty = bars + 2 * STAGES + 2;    // [2]       epilogue -> MMA (8 warp arrivals)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = GATEUP ? a.H : a.I;
    const int KB = K / BK;
    const int MT = (GATEUP ? 2 * a.I : a.H) / BM;                 // m-tiles of the packed matrix
    const size_t w13_bytes = matrix_bytes(2 * a.I, a.H);
    const int total_tiles = (*a.n_tiles) * MT;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 9);           // the 8 A-producer warps of this k-half + the TMA thread's expect_tx arrive
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ MMA issuer
        // ONE thread runs the loop (the other lanes wait at the warp barrier below).  tcgen05.mma issue blocks while
        // the tensor pipe is busy, and the pipe holds little beyond the MMA it executes: every instruction this
        // thread spends between two MMAs is time the pipe may drain, and with six busy warps on the same scheduler
        // each instruction takes many cycles to issue (measured alone: the same four MMAs per stage run at N / 2
        // cycles each with compile-time operands, at 150-160 cycles each, whatever N, behind run-time ring
        // arithmetic and a barrier test).  So the ring is unrolled (stage index, barrier addresses and operand offsets
        // are compile-time constants) and the NEXT stage's barrier is tested before this stage's MMAs are issued,
        // the answer being read after them.  Shapes whose stage count per tile is not a multiple of the ring depth
        // take the plain loop.
        PROF_DECL;
        if (lane == 0) {
            int tcount = 0;
            bool ok = true;
            const uint64_t da0 = make_desc_a(smem_u32(sA)), db0 = make_desc_b(smem_u32(sB));
            if ((2 * KB) % STAGES == 0) {
                int ph = 0;                                        // parity of the ring's current turn
                bool ready = false;                                // next stage's barrier already seen complete
                for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tcount) {
                    const Tile tl = a.tiles[t / MT];
                    const int n_mma = (tl.nrows + 15) & ~15;
                    const uint32_t idesc = make_idesc(n_mma);
                    const int buf = tcount & 1;
                    if (!mbar_try(&acc_empty[buf], ((tcount >> 1) & 1) ^ 1)) {
                        PROF_WAIT_BEGIN;
                        ok = mbar_wait(&acc_empty[buf], ((tcount >> 1) & 1) ^ 1, abort_flag, a.status);
                        PROF_WAIT_END;
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * BN_T;
                    for (int ks0 = 0; ks0 < 2 * KB && ok; ks0 += STAGES) {
#pragma unroll
                        for (int st = 0; st < STAGES; ++st) {
                            if (!ready) {
                                PROF_WAIT_BEGIN;
                                ok = mbar_wait(&full[st], ph, abort_flag, a.status);
                                PROF_WAIT_END;
                                if (!ok) break;
                            }
                            const int nst = (st + 1) % STAGES;
                            const bool ready_next = mbar_try(&full[nst], nst ? ph : ph ^ 1);
                            const uint64_t da = da0 + (uint64_t)(st * (A_STAGE_BYTES >> 4));
                            const uint64_t db = db0 + (uint64_t)(st * (B_STAGE_BYTES >> 4));
#pragma unroll
                            for (int j = 0; j < BKS / 16; ++j)     // K16 step j: A two k-chunks on, B 32 bytes on
                                tc_mma(d_tmem, da + (uint64_t)(j * 2 * A_LBO >> 4), db + (uint64_t)((j * 32) >> 4), idesc, (ks0 | st | j) ? 1u : 0u);
                            tc_commit(&empty[st]);                 // stage reusable once these MMAs have read it
                            ready = ready_next;
                        }
                        ph ^= 1;
                    }
                    if (ok) tc_commit(&acc_full[buf]);             // accumulator complete
                }
            } else {
                int s = 0, ph = 0;                                 // ring position of the next stage to consume
                for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tcount) {
                    const Tile tl = a.tiles[t / MT];
                    const int n_mma = (tl.nrows + 15) & ~15;
                    const uint32_t idesc = make_idesc(n_mma);
                    const int buf = tcount & 1;
                    ok = mbar_wait(&acc_empty[buf], ((tcount >> 1) & 1) ^ 1, abort_flag, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * BN_T;
                    for (int ks = 0; ks < 2 * KB; ++ks) {
                        if (!mbar_try(&full[s], ph)) ok = mbar_wait(&full[s], ph, abort_flag, a.status);
                        if (!ok) break;
                        const uint64_t da = da0 + (uint64_t)(s * (A_STAGE_BYTES >> 4));
                        const uint64_t db = db0 + (uint64_t)(s * (B_STAGE_BYTES >> 4));
#pragma unroll
                        for (int j = 0; j < BKS / 16; ++j)
                            tc_mma(d_tmem, da + (uint64_t)(j * 2 * A_LBO >> 4), db + (uint64_t)((j * 32) >> 4), idesc, (ks | j) ? 1u : 0u);
                        tc_commit(&empty[s]);
                        if (++s == STAGES) { s = 0; ph ^= 1; }
                    }
                    if (ok) tc_commit(&acc_full[buf]);
                }
            }
        }
        __syncwarp();
        PROF_REPORT("mma");
    } else if ((warp >= 4 && warp < 8) || (warp >= 16 && warp < 20)) {
        // ------------------------------------------------------------------ epilogue
        const int e = warp & 3;                                    // TMEM lane quarter
        const int odd = warp >= 16 ? 32 : 0;                       // second group takes the odd 32-column chunks
        int tcount = 0;
        bool ok = true;
        PROF_DECL;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tcount) {
            const Tile tl = a.tiles[t / MT];
            const int mt = t % MT;
            const int buf = tcount & 1;
            constexpr int CHUNKS = (BN_T + 63) / 64;               // 32-column chunks of this warp in a full tile
            const EpiloguePre<CHUNKS> pre = epilogue_prefetch<GATEUP, CHUNKS>(a, tl, odd, lane, offsets, topk_w);
            PROF_WAIT_BEGIN;
            ok = mbar_wait(&acc_full[buf], (tcount >> 1) & 1, abort_flag, a.status);
            PROF_WAIT_END;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            epilogue_tile<GATEUP, CHUNKS>(a, tl, mt, e, odd, lane, tmem_base + buf * BN_T, pre, act_out, y_out);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
        PROF_REPORT("epilogue");
    } else if (warp == 1) {
        // ------------------------------------------------------------------ B producer (TMA, one thread issues)
        int s = 0, ph = 0;
        bool ok = true;
        PROF_DECL;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const Tile tl = a.tiles[t / MT];
            const int row0 = offsets[tl.key] + tl.n0;
            const int n_mma = (tl.nrows + 15) & ~15;               // rows of the box = rows the MMAs read
            const CUtensorMap* map = maps + (n_mma / 16 - 1);
            for (int ks = 0; ks < 2 * KB; ++ks) {
                {
                    PROF_WAIT_BEGIN;
                    ok = mbar_wait(&empty[s], ph ^ 1, abort_flag, a.status);
                    PROF_WAIT_END;
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane == 0) {
                    mbar_expect_tx(&full[s], n_mma * 128);
                    tma_load_2d(smem_u32(sB + s * B_STAGE_BYTES), map, ks * BKS, row0, &full[s]);
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; ph ^= 1; }
            }
        }
        PROF_REPORT("B producer");
    } else if (warp >= 8 && !(warp >= 16 && warp < 20)) {
        // ------------------------------------------------------------------ A producers (dequantise)
        // A warp converts WHOLE packed blocks of one 16-row panel: both 64-wide halves, that is two consecutive ring
        // stages, with the block's scales split once (converting one half per warp, each half's warp split the same
        // scales and paid the loop's fixed instructions per 64 of K: these warps bound the kernel).  Warps 8-15 take
        // the even blocks of the CTA's block stream, warps 20-27 the odd ones.
        const int pw = warp & 7;                                   // panel of the tile = 8-row groups 2*pw, 2*pw+1
        const int par = warp >= 20 ? 1 : 0;                        // parity of this warp's blocks in the CTA's block stream
        const int q = lane >> 2, c = lane & 3;
        bool ok = true;
        PROF_DECL;
        // The conversion side needs nothing of a tile but its weights, so the warp walks ONE stream of blocks over all
        // of the CTA's tiles, its loads one of its blocks (two of the stream) ahead of the conversion ACROSS tile
        // boundaries.  The load cursor knows its tile's key one tile early, so entering a tile costs no dependent load.
        const int my_tiles = blockIdx.x < total_tiles ? (total_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
        const int total_blocks = my_tiles * KB;                    // of the stream; this warp converts par, par + 2, ...
        auto panel_row = [&](int t, int key) -> const uint8_t* {
            const uint8_t* mat = a.slots + (size_t)(key % a.num_slots) * a.slot_stride + (GATEUP ? 0 : w13_bytes);
            return mat + (size_t)((t % MT) * 8 + pw) * KB * kBlockBytes + lane * 16;
        };
        int c_t = blockIdx.x, c_kb = par, c_g = par;               // load cursor: tile, block of it, index in the stream
        int c_key_next = 0;
        const uint8_t* c_pn = nullptr;
        auto enter_tiles = [&]() {                                 // bring the cursor's block index back inside a tile
            while (c_kb >= KB && c_t < total_tiles) {
                c_kb -= KB;
                c_t += gridDim.x;
                if (c_t < total_tiles) {
                    c_pn = panel_row(c_t, c_key_next);
                    if (c_t + (int)gridDim.x < total_tiles) c_key_next = a.tiles[(c_t + gridDim.x) / MT].key;
                }
            }
        };
        if (my_tiles) {
            c_pn = panel_row(c_t, a.tiles[c_t / MT].key);
            if (c_t + (int)gridDim.x < total_tiles) c_key_next = a.tiles[(c_t + gridDim.x) / MT].key;
            enter_tiles();                                         // KB == 1 and par == 1: the first block is the next tile's
        }
        constexpr int PF = 2;                                      // blocks in flight per lane (this one + 1 ahead)
        uint4 w[PF][2];
        uint32_t sc[PF];
        auto fetch = [&](uint4 (&wv)[2], uint32_t& sv) {           // request the cursor's block, move the cursor two on
            const uint8_t* blk = c_pn + (size_t)c_kb * kBlockBytes;
            wv[0] = ldg_stream128(blk);
            wv[1] = ldg_stream128(blk + 512);
            sv = ldg_stream32(blk - lane * 16 + kCodeBytes + q * 4);
            c_g += 2;
            c_kb += 2;
            enter_tiles();
        };
        if (c_g < total_blocks) fetch(w[0], sc[0]);
        // Stage index of (block g, half h) = 2 g + h; this warp's blocks are g = par + 2 i, so the stage count is
        // n = 2 par + 4 i + h.  With the ring depth a power of two (4 or 8) and the loop unrolled by two blocks, the ring
        // position of (u = i mod 2, h) is loop-invariant: ((2 par + 4 u) mod STAGES) + h.  Store addresses and barrier
        // addresses are therefore formed once, outside the loop (the address arithmetic of a run-time ring position was a
        // tenth of this loop's instructions).
        static_assert(STAGES == 4 || STAGES == 8, "ring positions of the conversion warps are precomputed for these depths");
        constexpr int LOG_STAGES = STAGES == 4 ? 2 : 3;
        unsigned char* stage_ptr[2];
        uint64_t* full_ptr[2];
        uint64_t* empty_ptr[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int sb = (2 * par + 4 * u) & (STAGES - 1);
            stage_ptr[u] = sA + sb * A_STAGE_BYTES + (2 * pw) * A_SBO + c * A_LBO + q * 16;
            full_ptr[u] = &full[sb];
            empty_ptr[u] = &empty[sb];
        }
        int n = 2 * par;                                           // stage count of the next block's first half
        for (int g0 = par; g0 < total_blocks && ok; g0 += 2 * PF) {
#pragma unroll
            for (int u = 0; u < PF; ++u) {
                if (g0 + 2 * u >= total_blocks) break;
                if (c_g < total_blocks) fetch(w[(u + 1) % PF], sc[(u + 1) % PF]);       // keep one block in flight
                const __half2 sh = *reinterpret_cast<const __half2*>(&sc[u]);
                const ScaleSplit s_lo = split_scale(__low2float(sh));                 // row q
                const ScaleSplit s_hi = split_scale(__high2float(sh));                // row q + 8
                const uint32_t ph = (n >> LOG_STAGES) & 1;                            // the same for both halves
#pragma unroll
                for (int h = 0; h < 2; ++h) {                                         // the block's two halves = two stages
                    {
                        PROF_WAIT_BEGIN;
                        ok = mbar_wait(empty_ptr[u] + h, ph ^ 1, abort_flag, a.status);
                        PROF_WAIT_END;
                    }
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    unsigned char* dst = stage_ptr[u] + h * A_STAGE_BYTES;
                    const uint32_t words[4] = {w[u][h].x, w[u][h].y, w[u][h].z, w[u][h].w};
#pragma unroll
                    for (int wi = 0; wi < 4; ++wi) {
                        const int r = wi & 1, set = wi >> 1;
                        const uint4 val = dequant_word(words[wi], r ? s_hi : s_lo);
                        *reinterpret_cast<uint4*>(dst + r * A_SBO + 4 * set * A_LBO) = val;   // k-chunk 4 set + c of row group 2 pw + r
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full_ptr[u] + h);
                }
                if (!ok) break;
                n += 4;
            }
        }
        PROF_REPORT("A producer");
    }

    // ---------------------------------------------------------------------- teardown (all roles, abort or not)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing will ever complete, with a short
// budget; the wait must give up, raise the abort flag and the status word, and the kernel must return normally.
__global__ void wait_timeout_selftest_kernel(int* status, long long budget, int* result) {
    __shared__ uint64_t bar;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait(&bar, 0, &abort_word, status, budget);     // phase 0 never completes
    __syncthreads();
    if (threadIdx.x == 0) *result = (ok ? 0 : 1) | (abort_word ? 2 : 0);
}

// n-tiles of one wave: every active group is cut into balanced runs of at most `bn` grouped rows (multiples of 16).
// Executed by one whole CTA (any multiple of 32 threads up to 1024): thread g handles group g, an exclusive scan of
// the piece counts places its tiles.
__device__ void build_tile_list(const int32_t* __restrict__ counts, const int32_t* __restrict__ group_keys,
                                const int32_t* __restrict__ wave_start, Tile* __restrict__ tiles,
                                int32_t* __restrict__ n_tiles, int bn) {
    __shared__ int s_warp[32];
    __shared__ int s_running;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x, nwarp = nthr >> 5;
    const int g0 = wave_start[0], ng = wave_start[1] - g0;
    if (tid == 0) s_running = 0;
    __syncthreads();
    for (int base = 0; base < ng; base += nthr) {
        const int g = base + tid;
        int key = 0, cnt = 0, pieces = 0, per = 0;
        if (g < ng) {
            key = group_keys[g0 + g];
            cnt = counts[key];
            pieces = (cnt + bn - 1) / bn;
            per = ((cnt + pieces - 1) / pieces + 15) & ~15;
            pieces = (cnt + per - 1) / per;
        }
        int incl = pieces;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int wbase = 0, total = 0;
        for (int w = 0; w < nwarp; ++w) {
            if (w < warp) wbase += s_warp[w];
            total += s_warp[w];
        }
        int pos = s_running + wbase + incl - pieces;
        for (int n0 = 0; n0 < cnt; n0 += per) tiles[pos++] = Tile{key, n0, min(per, cnt - n0), 0};
        __syncthreads();
        if (tid == 0) s_running += total;
        __syncthreads();
    }
    if (tid == 0) *n_tiles = s_running;
}

__global__ void __launch_bounds__(1024)
tile_list_kernel(const int32_t* __restrict__ counts, const int32_t* __restrict__ group_keys,
                 const int32_t* __restrict__ wave_start, Tile* __restrict__ tiles, int32_t* __restrict__ n_tiles, int bn) {
    build_tile_list(counts, group_keys, wave_start, tiles, n_tiles, bn);
}

// grouped copy of the hidden states: row r of the plan order = hidden row of token perm[r] / k
// CTA 0 also builds the tile list of the call's only wave when `tiles` is given (one launch less).
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16* __restrict__ hidden, const int32_t* __restrict__ perm,
                   const int32_t* __restrict__ n_valid, int top_k, int H, __nv_bfloat16* __restrict__ xg,
                   const int32_t* __restrict__ counts, const int32_t* __restrict__ group_keys,
                   const int32_t* __restrict__ wave_start, Tile* __restrict__ tiles, int32_t* __restrict__ n_tiles, int bn) {
    if (blockIdx.x == 0 && tiles) build_tile_list(counts, group_keys, wave_start, tiles, n_tiles, bn);
    // one warp per row, eight rows per CTA; a lane keeps up to eight 16-byte loads in flight before it stores
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 8 + warp;
    if (r >= *n_valid) return;
    int token = 0;
    if (lane == 0) token = perm[r] / top_k;
    token = __shfl_sync(0xffffffffu, token, 0);
    const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)token * H);
    uint4* dst = reinterpret_cast<uint4*>(xg + (size_t)r * H);
    const int n16 = H / 8;
    for (int base = 0; base < n16; base += 256) {
        uint4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = base + lane + 32 * j;
            if (i < n16) v[j] = src[i];
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = base + lane + 32 * j;
            if (i < n16) dst[i] = v[j];
        }
    }
}

}  // namespace

size_t prefill_scratch_bytes(int max_pairs, int num_experts) {
    return ((size_t)max_pairs / 16 + num_experts + 16) * sizeof(Tile) + 256;
}

static_assert(sizeof(CUtensorMap) == 128, "PrefillMaps mirrors CUtensorMap objects");

// 2-D row-major BF16 matrix [rows, cols] -> tensor map with a 64-column x `box_rows`-row box, 128-byte swizzle
static int encode_map(CUtensorMap* out, const void* base, int rows, int cols, int box_rows) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess || !p) return EXMOE_ERR_CUDA;
        fn = reinterpret_cast<EncodeFn>(p);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult rc = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int prefill_setup(PrefillMaps* maps, const __nv_bfloat16* xg, const __nv_bfloat16* act, int max_pairs, int H, int I) {
    static_assert(kPrefillMapBytes == 2 * N_MAPS * sizeof(CUtensorMap), "map families of the two operands");
    alignas(64) CUtensorMap host[2 * N_MAPS];
    int rc = EXMOE_OK;
    for (int i = 0; i < N_MAPS && !rc; ++i) {
        rc = encode_map(&host[i], xg, max_pairs, H, 16 * (i + 1));
        if (!rc) rc = encode_map(&host[N_MAPS + i], act, max_pairs, I, 16 * (i + 1));
    }
    if (!rc && cudaMemcpy(maps->dev, host, sizeof(host), cudaMemcpyHostToDevice) != cudaSuccess) rc = EXMOE_ERR_CUDA;
    return rc;
}

void launch_wait_selftest(int* status, long long budget_cycles, int* result, cudaStream_t st) {
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(status, budget_cycles, result);
    count_launch();
}

void launch_gather_rows(const __nv_bfloat16* hidden, const int32_t* perm, const int32_t* n_valid, int n_pairs, int top_k,
                        int H, __nv_bfloat16* xg, const GemmArgs* single_wave, const int32_t* wave_start, void* scratch,
                        bool small_n, cudaStream_t st) {
    int32_t* n_tiles = reinterpret_cast<int32_t*>(scratch);
    Tile* tiles = single_wave ? reinterpret_cast<Tile*>(reinterpret_cast<unsigned char*>(scratch) + 256) : nullptr;
    gather_rows_kernel<<<(n_pairs + 7) / 8, 256, 0, st>>>(hidden, perm, n_valid, top_k, H, xg, single_wave ? single_wave->counts : nullptr,
                                                 single_wave ? single_wave->group_keys : nullptr, wave_start, tiles, n_tiles,
                                                 small_n ? BN_SMALL : BN);
    count_launch();
}

// One wave of the tensor-core path: tile list, gate/up GEMM + SwiGLU, down GEMM x routing weight.
void launch_prefill_wave(const GemmArgs& g, const int32_t* wave_start, void* scratch, int* status, const PrefillMaps* maps,
                         __nv_bfloat16* act, const float* topk_w, float* y, int which, bool small_n, cudaStream_t st) {
    int32_t* n_tiles = reinterpret_cast<int32_t*>(scratch);
    Tile* tiles = reinterpret_cast<Tile*>(reinterpret_cast<unsigned char*>(scratch) + 256);
    PrefillArgs a{};
    a.slots = g.slots;
    a.slot_stride = g.slot_stride;
    a.perm = g.perm;
    a.tiles = tiles;
    a.n_tiles = n_tiles;
    a.num_slots = g.num_slots;
    a.top_k = g.top_k;
    a.H = g.H;
    a.I = g.I;
    a.status = status;
    constexpr int kStagesLarge = 4, kStagesSmall = 8;
    const size_t smem_large = (size_t)kStagesLarge * (A_STAGE_BYTES + BN * 128) + 256 + 1024;
    const size_t smem_small = (size_t)kStagesSmall * (A_STAGE_BYTES + BN_SMALL * 128) + 256 + 1024;
    static SmemOnce once[4];
    allow_smem(prefill_gemm_kernel<true, BN, kStagesLarge>, (int)smem_large, once[0]);
    allow_smem(prefill_gemm_kernel<false, BN, kStagesLarge>, (int)smem_large, once[1]);
    allow_smem(prefill_gemm_kernel<true, BN_SMALL, kStagesSmall>, (int)smem_small, once[2]);
    allow_smem(prefill_gemm_kernel<false, BN_SMALL, kStagesSmall>, (int)smem_small, once[3]);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const CUtensorMap* mx = reinterpret_cast<const CUtensorMap*>(maps->dev);
    const CUtensorMap* ma = mx + N_MAPS;
    if (which & 4) {
        tile_list_kernel<<<1, 1024, 0, st>>>(g.counts, g.group_keys, wave_start, tiles, n_tiles, small_n ? BN_SMALL : BN);
        count_launch();
    }
    if (which & 1) {
        if (small_n)
            prefill_gemm_kernel<true, BN_SMALL, kStagesSmall><<<sms, NUM_THREADS, smem_small, st>>>(a, mx, act, nullptr, g.offsets, nullptr);
        else
            prefill_gemm_kernel<true, BN, kStagesLarge><<<sms, NUM_THREADS, smem_large, st>>>(a, mx, act, nullptr, g.offsets, nullptr);
        count_launch();
    }
    if (which & 2) {
        if (small_n)
            prefill_gemm_kernel<false, BN_SMALL, kStagesSmall><<<sms, NUM_THREADS, smem_small, st>>>(a, ma, nullptr, topk_w, g.offsets, y);
        else
            prefill_gemm_kernel<false, BN, kStagesLarge><<<sms, NUM_THREADS, smem_large, st>>>(a, ma, nullptr, topk_w, g.offsets, y);
        count_launch();
    }
}

}  // namespace exmoe
