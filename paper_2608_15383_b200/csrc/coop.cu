// One-launch one-token layer: both grouped GEMMs of Section 3.4 and the sum of Eq. 2 in ONE cooperative kernel whose
// CTAs are all resident (one per SM) and meet once, at a bounded device-wide barrier between the two projections.
//
// A decode step is bound by latency, not by bandwidth: two dependent launches that each read ids, then weights, then
// compute leave HBM idle for most of the step.  Here every weight byte of the step is requested in the first
// instructions of the one launch:
//   * gate/up: CTA (s, p) owns a slice of pair p's intermediates (as many panel pairs as its 16 warps hold in
//     registers, one (panel pair, K range) unit per warp, loaded block by block two blocks ahead of the arithmetic);
//   * down: CTA number L owns output panel(s) L*dp .. of EVERY pair: their packed blocks follow the gate/up loads on
//     the same request path (cp.async into shared memory), so they are in flight or there when the barrier opens;
//   * after gate/up + SwiGLU the CTA publishes its BF16 activations (global memory) and arrives at the barrier
//     (one acquire-release atomic; the last arriver flips a generation word, the others poll it with a bounded wait);
//   * then every CTA reads all pairs' activation rows (L2), runs its down units (one (pair, K range) unit per chain,
//     the K ranges the other decode kernels use), and adds ranges, routing weights and the k pair rows in the fixed
//     order j = 0..k-1 in shared memory: no partial results ever go to global memory and nothing follows the sum.
// Co-residency is what makes waiting legal: the launch is cooperative (it fails, and the caller falls back, if the
// CTAs cannot all be resident).  Arithmetic, K ranges and summation orders are those of decode.cu: same bits.
#include "common.cuh"
#include "frag.cuh"
#include "mbar.cuh"
#include "chain.cuh"

#include <cstdio>
#include <mutex>

#ifndef EXMOE_COOP_ABLATE
#define EXMOE_COOP_ABLATE 0
#endif

namespace exmoe {

namespace {

constexpr int kCoThreads = 512;
constexpr int kCoWarps = kCoThreads / 32;
constexpr int kCoSmemLimit = 225 * 1024;
constexpr int kCoMaxPairs = 32;

struct CoopArgs {
    const uint8_t* slots;
    size_t slot_stride;
    size_t w13_bytes;
    const int32_t* ids;
    const int32_t* slot_of;                          // null: slot = expert id (C = E)
    const __nv_bfloat16* hidden;
    const float* topk_w;
    __nv_bfloat16* act;                              // [T*k, I] SwiGLU activations, pair order (the exchange buffer)
    __nv_bfloat16* out;                              // [T, H]
    int* sync;                                       // [0] arrivals of the running launch, [1] generation; zero-initialised
    int* status;
    int32_t* saved_ids;
    int E, k, H, I, n_pairs;
    int bpw_g, ks_g_log2, bpw_d, ks_d;               // blocks per K range / ranges, gate/up and down
    int npp;                                         // panel pairs per CTA (gate/up)
    int dp;                                          // output panels per CTA (down)
    int n_cta;
};

__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

#ifdef EXMOE_COOP_PROF
__device__ __forceinline__ unsigned long long gtime() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define CO_PROF(i) if (threadIdx.x == 0) prof_t[i] = gtime();
#else
#define CO_PROF(i)
#endif

template <int NBG>
__global__ void __launch_bounds__(kCoThreads, 1)
coop_decode_kernel(CoopArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
#ifdef EXMOE_COOP_PROF
    unsigned long long prof_t[10] = {};
    CO_PROF(0)
#endif
    // grid = (gate/up slices per pair, pairs)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int p = blockIdx.y, L = blockIdx.y * gridDim.x + blockIdx.x;
    const int P = a.n_pairs, KBg = a.H / kGroup, KBd = a.I / kGroup;
    const int Ug = a.npp << a.ks_g_log2;
    const int panels = a.H / kPanelRows;
    const int d0 = L * a.dp, nd = max(0, min(a.dp, panels - d0));                // this CTA's output panels [d0, d0 + nd)
    const int Ud = nd * P * a.ks_d;                                              // down units: ((d * P + pair) * ks_d + range)
    const uint32_t dn_unit_bytes = (uint32_t)a.bpw_d * kBlockBytes;

    unsigned char* wdn = smem;                                                   // [dp * P * ks_d][range]
    unsigned char* xs = wdn + (size_t)a.dp * P * a.ks_d * dn_unit_bytes;         // per-warp K ranges of the hidden row
    unsigned char* as = xs + (size_t)kCoWarps * NBG * kGroup * 2;                // [P][I] activations of all pairs
    float* adj_d = reinterpret_cast<float*>(as + (size_t)P * a.I * 2);           // [P][KBd]
    float* red_g = adj_d + (size_t)P * KBd;                                      // [Ug][2][16]
    float* part = red_g + (size_t)Ug * 32;                                       // [dp * P * ks_d][16]
    float* s_rw = part + (size_t)a.dp * P * a.ks_d * 16;                         // [P]
    int* s_slot = reinterpret_cast<int*>(s_rw + P);                              // [P] slot of the pair, -1 = invalid id
    int* s_flag = s_slot + P;                                                    // [0] barrier outcome

#if EXMOE_COOP_ABLATE == 7
    return;                                             // timing only: the launch itself
#endif
    // Loads that do not depend on the ids go first: this warp's K range of the hidden row.
    const int t = p / a.k;
    const unsigned char* xrow_g = reinterpret_cast<const unsigned char*>(a.hidden + (size_t)t * a.H);
    const int my_pp = warp >> a.ks_g_log2, my_ks = warp & ((1 << a.ks_g_log2) - 1);
    constexpr int XL = (NBG * 16 + 31) / 32;                                     // 16-byte chunks of the row per lane
    uint4 xpre[XL];
#pragma unroll
    for (int i = 0; i < XL; ++i) {
        xpre[i] = make_uint4(0, 0, 0, 0);
        if (i * 32 + lane < NBG * 16) xpre[i] = ldg_early128(xrow_g + ((size_t)my_ks * NBG * 16 + i * 32 + lane) * 16);
    }
    const int id = a.ids[p];
    int gen0 = 0;
    if (tid == 0) gen0 = ld_acquire(a.sync + 1);                                 // before this CTA arrives, so before any flip
    // the slots of all pairs (the down units of this CTA span every pair), their routing weights
    if (tid < P) {
        const int v = a.ids[tid];
        const bool okv = (unsigned)v < (unsigned)a.E;
        s_slot[tid] = okv ? (a.slot_of ? a.slot_of[v] : v) : -1;
        s_rw[tid] = a.topk_w[tid];
        if (L == 0) {                                                            // keep the ids (plan on request), flag bad ones
            a.saved_ids[tid] = v;
            if (!okv) atomicExch(a.status, EXMOE_ERR_BAD_EXPERT_ID);
        }
    }
    const bool id_ok = (unsigned)id < (unsigned)a.E;
    const int slot = id_ok ? (a.slot_of ? a.slot_of[id] : id) : 0;
    const uint8_t* wbase = a.slots + (size_t)slot * a.slot_stride;
    const size_t pp0 = (size_t)blockIdx.x * a.npp;                               // first panel pair of this CTA
    __syncthreads();                                                             // s_slot
    CO_PROF(1)

    // ---- gate/up: this warp's unit goes straight into registers, block by block, two blocks ahead of the arithmetic
    // (a warp that has issued everything first sits out the load queue's back-pressure with nothing to compute); its
    // part of the hidden row goes into its own piece of shared memory; adjv[b] = -136 * (block sum), formed as the
    // staging loops of the other decode kernels form it.  The warp's down units follow on the same path.
    uint4 wreg[NBG][2][2];
    uint32_t sreg[NBG][2];
    float adjv[NBG];
    unsigned char* xw = xs + (size_t)warp * NBG * kGroup * 2;
    const bool has_unit = id_ok && warp < Ug;
    const uint8_t* gu_base = wbase + (2 * (pp0 + my_pp) * KBg + (size_t)my_ks * NBG) * kBlockBytes;
    auto issue_block = [&](int b) {
        if (!has_unit) return;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const uint8_t* blk = gu_base + ((size_t)m * KBg + b) * kBlockBytes;
            wreg[b][m][0] = ldg_stream128(blk + lane * 16);
            wreg[b][m][1] = ldg_stream128(blk + 512 + lane * 16);
            sreg[b][m] = ldg_stream32(blk + kCodeBytes + q * 4);
        }
    };
    auto issue_down = [&]() {
        for (int u = warp; u < Ud; u += kCoWarps) {
            const int r = u % a.ks_d, dq = u / a.ks_d, pr = dq % P, d = dq / P;
            const int sl = s_slot[pr];
            if (sl < 0) continue;
            const uint8_t* src = a.slots + (size_t)sl * a.slot_stride + a.w13_bytes +
                                 (((size_t)d0 + d) * KBd + (size_t)r * a.bpw_d) * kBlockBytes;
            unsigned char* dst = wdn + (size_t)u * dn_unit_bytes;
            for (uint32_t off = lane * 16; off < dn_unit_bytes; off += 32 * 16) cp_async16(dst + off, src + off);
        }
    };
#ifdef EXMOE_COOP_UPFRONT
#pragma unroll
    for (int b = 0; b < NBG; ++b) issue_block(b);
    issue_down();
#else
    issue_block(0);
    if (NBG > 1) issue_block(1);
    if (NBG <= 2) issue_down();
#endif
#pragma unroll
    for (int i = 0; i < XL; ++i) {
        const int ck = i * 32 + lane;
        if (ck < NBG * 16) *reinterpret_cast<uint4*>(xw + ck * 16) = xpre[i];
        float sx = sum8_bf16(xpre[i]);
#pragma unroll
        for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
        const float lo = __shfl_sync(0xffffffffu, sx, 0), hi = __shfl_sync(0xffffffffu, sx, 16);
        // __fmul_rn: the product is rounded on its own, as where the other kernels keep it in shared memory
        // (left to the compiler it would be contracted into the accumulator addition that uses it)
        if (2 * i < NBG) adjv[2 * i] = __fmul_rn(-136.f, lo);
        if (2 * i + 1 < NBG) adjv[2 * i + 1] = __fmul_rn(-136.f, hi);
    }
    __syncwarp();
    float tot[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
    for (int b = 0; b < NBG; ++b) {
#ifndef EXMOE_COOP_UPFRONT
        if (b + 2 < NBG) issue_block(b + 2);
        if (NBG > 2 && b + 3 == NBG) issue_down();      // behind the last gate/up block
#endif
#if EXMOE_COOP_ABLATE == 5 || EXMOE_COOP_ABLATE == 6
        if (has_unit) { tot[0][0] += __uint_as_float(wreg[b][0][0].x ^ wreg[b][0][1].y ^ wreg[b][1][0].z ^ wreg[b][1][1].w ^ sreg[b][0] ^ sreg[b][1]); }   // timing only: loads without arithmetic
#else
        if (has_unit) chain_block_regs(wreg[b], sreg[b], adjv[b], b, xw, lane, tot);
#endif
    }
#if EXMOE_COOP_ABLATE == 6
    cp_async_wait_all();
    if (tot[0][0] == 123.f) a.out[0] = __float2bfloat16_rn(tot[0][0]);
    return;                                             // timing only: ids, all loads, no arithmetic (with ABLATE 5's fold)
#endif
    if (has_unit && c == 0) {
        float* r = red_g + (size_t)warp * 32;
        r[q] = tot[0][0];
        r[q + 8] = tot[0][1];
        r[16 + q] = tot[1][0];
        r[16 + q + 8] = tot[1][1];
    }
    __syncthreads();
    CO_PROF(2)
    // K ranges added in ascending order, SwiGLU, one rounding to BF16; published for every CTA
    if (id_ok)
        for (int i = tid; i < a.npp * kPanelRows; i += kCoThreads) {
            const int pp = i >> 4, r = i & 15;
            const float* base = red_g + ((size_t)pp << a.ks_g_log2) * 32;
            float g = base[r], u = base[16 + r];
            for (int s = 1; s < (1 << a.ks_g_log2); ++s) {
                g += base[s * 32 + r];
                u += base[s * 32 + 16 + r];
            }
            a.act[(size_t)p * a.I + pp0 * kPanelRows + i] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * u);
        }
    __syncthreads();

    CO_PROF(3)
#if EXMOE_COOP_ABLATE == 1
    cp_async_wait_all();
    return;                                             // timing only: up to the published activations
#endif
    // ---- the one meeting point: every CTA's activations are published before any CTA reads them
    if (tid == 0) {
        int old;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(a.sync) : "memory");
        int okb = 1;
        if (old == a.n_cta - 1) {
            a.sync[0] = 0;                              // ready for the next launch
            asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(a.sync + 1), "r"(gen0 + 1) : "memory");
        } else {
            const long long t0 = clock64();
            while (ld_acquire(a.sync + 1) == gen0) {
                if (clock64() - t0 > kWaitBudget) {     // bounded: report and leave, nothing is written
                    atomicExch(a.status, EXMOE_ERR_TIMEOUT);
                    okb = 0;
                    break;
                }
            }
        }
        s_flag[0] = okb;
    }
    __syncthreads();
    cp_async_wait_all();                                // this lane's pieces of the warp's down units ...
    __syncwarp();                                       // ... and the other lanes'
    if (!s_flag[0]) return;
    CO_PROF(4)
#if EXMOE_COOP_ABLATE == 2
    return;                                             // timing only: up to the opened barrier
#endif

    // ---- all pairs' activation rows (written by other SMs: read through L2), their block corrections
    for (int i = tid; i < P * a.I / 8; i += kCoThreads)
        *reinterpret_cast<uint4*>(as + (size_t)i * 16) = __ldcg(reinterpret_cast<const uint4*>(a.act) + i);
    __syncthreads();
    block_sums(as, P * a.I / 8, adj_d, warp, lane, kCoThreads);
    __syncthreads();
    CO_PROF(5)
#if EXMOE_COOP_ABLATE == 3
    return;                                             // timing only: up to the staged activations
#endif

    // ---- down: one (panel, pair, K range) unit per chain, two chains at a time
    for (int u = warp; u < Ud; u += 2 * kCoWarps) {
        const int u2 = u + kCoWarps;
        const int r1 = u % a.ks_d, pr1 = (u / a.ks_d) % P;
        const bool v1 = s_slot[pr1] >= 0;
        bool v2 = false;
        int r2 = 0, pr2 = 0;
        if (u2 < Ud) {
            r2 = u2 % a.ks_d;
            pr2 = (u2 / a.ks_d) % P;
            v2 = s_slot[pr2] >= 0;
        }
        if (v1 && v2) {
            const unsigned char* const w[2] = {wdn + (size_t)u * dn_unit_bytes, wdn + (size_t)u2 * dn_unit_bytes};
            const unsigned char* const x[2] = {as + ((size_t)pr1 * a.I + (size_t)r1 * a.bpw_d * kGroup) * 2,
                                               as + ((size_t)pr2 * a.I + (size_t)r2 * a.bpw_d * kGroup) * 2};
            const float* const adj[2] = {adj_d + (size_t)pr1 * KBd + r1 * a.bpw_d, adj_d + (size_t)pr2 * KBd + r2 * a.bpw_d};
            float td[2][2];
            range_chain_rows<2>(w, a.bpw_d, x, adj, lane, td);
            if (c == 0) {
                part[(size_t)u * 16 + q] = td[0][0];
                part[(size_t)u * 16 + q + 8] = td[0][1];
                part[(size_t)u2 * 16 + q] = td[1][0];
                part[(size_t)u2 * 16 + q + 8] = td[1][1];
            }
        } else if (v1 || v2) {
            const int uu = v1 ? u : u2, rr = v1 ? r1 : r2, pr = v1 ? pr1 : pr2;
            const unsigned char* const w[1] = {wdn + (size_t)uu * dn_unit_bytes};
            const unsigned char* const x[1] = {as + ((size_t)pr * a.I + (size_t)rr * a.bpw_d * kGroup) * 2};
            const float* const adj[1] = {adj_d + (size_t)pr * KBd + rr * a.bpw_d};
            float td[1][2];
            range_chain_rows<1>(w, a.bpw_d, x, adj, lane, td);
            if (c == 0) {
                part[(size_t)uu * 16 + q] = td[0][0];
                part[(size_t)uu * 16 + q + 8] = td[0][1];
            }
        }
    }
    __syncthreads();
    CO_PROF(6)
#if EXMOE_COOP_ABLATE == 4
    return;                                             // timing only: everything but the final sum
#endif

    // ---- Eq. 2's sum: per pair the K ranges in ascending order, x routing weight, then the k pair rows in the order
    // j = 0..k-1 (products and sums rounded one by one, as where the other kernels keep them in memory)
    const int T = P / a.k;
    for (int i = tid; i < T * nd * kPanelRows; i += kCoThreads) {
        const int r16 = i & 15, d = (i >> 4) % nd, tt = (i >> 4) / nd;
        float sum = 0.f;
        for (int jj = 0; jj < a.k; ++jj) {
            const int pr = tt * a.k + jj;
            if (s_slot[pr] < 0) continue;
            const float* base = part + ((size_t)(d * P + pr) * a.ks_d) * 16 + r16;
            float res = base[0];
            for (int r = 1; r < a.ks_d; ++r) res = __fadd_rn(res, base[r * 16]);
            sum = __fadd_rn(sum, __fmul_rn(s_rw[pr], res));
        }
        a.out[(size_t)tt * a.H + (size_t)(d0 + d) * kPanelRows + r16] = __float2bfloat16_rn(sum);
    }
#ifdef EXMOE_COOP_PROF
    CO_PROF(7)
    if (tid == 0) {
        { const long long c0 = clock64(); while (clock64() - c0 < 100000) {} }
        printf("CO L=%d t0=%llu slots=%llu gu=%llu pub=%llu bar=%llu acts=%llu down=%llu end=%llu\n", L, prof_t[0], prof_t[1] - prof_t[0],
               prof_t[2] - prof_t[0], prof_t[3] - prof_t[0], prof_t[4] - prof_t[0], prof_t[5] - prof_t[0], prof_t[6] - prof_t[0],
               prof_t[7] - prof_t[0]);
    }
#endif
}

using CoopKernel = void (*)(CoopArgs);
CoopKernel coop_kernel(int nbg) {
    return nbg == 4 ? coop_decode_kernel<4> : nbg == 2 ? coop_decode_kernel<2> : coop_decode_kernel<1>;
}

}  // namespace

void decode_k_split(int K, int rows, bool down, int* ks, int* bpw);

// Launches the one-kernel layer when all of its CTAs can be resident at once; false = not taken (nothing queued).
bool launch_coop_decode(const GemmArgs& g, const SmallWave& w, int* sync_words, cudaStream_t st) {
#ifdef EXMOE_NO_COOP_DECODE
    return false;
#endif
    const int H = g.H, I = g.I, k = g.top_k, P = w.n_pairs;
    if (P < 1 || P > kCoMaxPairs || P > kCoopMaxPairs || P % k || !w.act || !sync_words) return false;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    int ks_g = 1, bpw_g = 1, ks_d = 1, bpw_d = 1;
    decode_k_split(H, I, false, &ks_g, &bpw_g);
    decode_k_split(I, H, true, &ks_d, &bpw_d);
    if (bpw_g != 1 && bpw_g != 2 && bpw_g != 4) return false;                   // the unit must fit a warp's registers
    int ks_g_log2 = 0;
    while ((1 << ks_g_log2) < ks_g) ++ks_g_log2;
    if ((1 << ks_g_log2) != ks_g || ks_g > kCoWarps) return false;
    const int pairs_total = I / kPanelRows;                                     // gate/up panel pairs of one expert
    int npp = kCoWarps >> ks_g_log2;
    while (npp > 1 && pairs_total % npp) npp >>= 1;
    const int gcta = pairs_total / npp, n_cta = gcta * P;
    const int panels = H / kPanelRows, dp = (panels + n_cta - 1) / n_cta;
    const size_t units = (size_t)dp * P * ks_d;
    const size_t smem = units * bpw_d * kBlockBytes + (size_t)kCoWarps * bpw_g * kGroup * 2 + (size_t)P * I * 2 +
                        (size_t)P * (I / kGroup) * 4 + (size_t)(npp * ks_g) * 32 * 4 + units * 16 * 4 + (size_t)P * 8 + 64;
    if (smem > (size_t)kCoSmemLimit) return false;

    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    CoopKernel kern = coop_kernel(bpw_g);
    static SmemOnce smem_once[3];
    if (!allow_smem(kern, kCoSmemLimit, smem_once[bpw_g == 4 ? 2 : bpw_g - 1])) {
        cudaGetLastError();
        return false;
    }
    // all CTAs resident at once, or not this path (per device: SM count x CTAs per SM for this kernel and footprint)
    static int sm_count[64] = {};
    if (!sm_count[dev] && cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kCoThreads, smem) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    if ((long long)per_sm * sm_count[dev] < n_cta) return false;

    CoopArgs a{};
    a.slots = g.slots;
    a.slot_stride = g.slot_stride;
    a.w13_bytes = matrix_bytes(2 * I, H);
    a.ids = w.ids;
    a.slot_of = w.slot_of;
    a.hidden = w.hidden;
    a.topk_w = w.topk_w;
    a.act = w.act;
    a.out = w.out;
    a.sync = sync_words;
    a.status = w.status;
    a.saved_ids = w.saved_ids;
    a.E = w.E;
    a.k = k;
    a.H = H;
    a.I = I;
    a.n_pairs = P;
    a.bpw_g = bpw_g; a.ks_g_log2 = ks_g_log2; a.bpw_d = bpw_d; a.ks_d = ks_d;
    a.npp = npp;
    a.dp = dp;
    a.n_cta = n_cta;

    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(gcta, P);
    lc.blockDim = dim3(kCoThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, kern, a) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    count_launch();
    return true;
}

}  // namespace exmoe
