// One-launch tiny-batch layer (T*k <= kSmallMaxPairs, one wave): both grouped GEMMs of Section 3.4 and the sum of
// Eq. 2 in ONE kernel, one small thread-block cluster per (token-expert pair, K range of the down projection).
//
// A decode step is bound by latency, not by bandwidth: two dependent launches that each read ids, then weights,
// then compute leave HBM idle for most of the step.  Here every byte the step needs is requested in the first
// instructions of the one launch, and no CTA ever waits for a CTA outside its own cluster:
//   * The down projection's K (the intermediate dimension) is cut into the K ranges whose partial sums the other
//     decode kernels add in ascending order (decode.cu: pick_cfg); range r covers intermediates
//     [r * 128 * bpw_d, (r + 1) * 128 * bpw_d).  A cluster of CS CTAs owns one pair and one range: it computes
//     exactly the SwiGLU activations that range needs, and nobody else needs them.
//   * CTA c of the cluster owns 1/CS of the range's intermediates (gate and up panels over the whole K of the
//     hidden state) and 1/CS of the output rows.  Both slices are brought into its shared memory with
//     cp.async.bulk copies (no multicast), one mbarrier per unit, so that a warp starts on a unit as soon as that
//     unit's bytes have landed.
//   * gate/up + SwiGLU for the CTA's intermediates; the BF16 activations go to the CTAs of the cluster through
//     distributed shared memory (st.async: the store completes transaction bytes on the receiver's mbarrier);
//   * the range's partial down projection of the CTA's output rows is written (unweighted) to a partial buffer;
//   * the CTA whose arrival completes a (token, 128-column slice) - arrival counter, no spin - forms every pair's
//     result as the ascending sum of its K ranges, multiplies by the routing weight and adds the k pair rows in the
//     order j = 0..k-1.
// Arithmetic, K ranges and summation orders are those of the pairwise and in-CTA-grouping kernels of decode.cu
// (same bits), so the layer output stays identical for every slot count and wave partition.
// Every wait is bounded (mbar.cuh); the cluster barrier is the hardware's (the CTAs of a cluster are co-scheduled
// and arrive unconditionally).  Cluster sizes stay small (4 at OLMoE's shape) because a B200 co-schedules 33
// clusters of 4 CTAs with ~210 KB of shared memory each but only 15 of 8 and 7 of 16.
#include "common.cuh"
#include "frag.cuh"
#include "mbar.cuh"
#include "chain.cuh"

#include <atomic>
#include <cstdio>
#include <mutex>

#ifndef EXMOE_CLUSTER_ABLATE
#define EXMOE_CLUSTER_ABLATE 0
#endif

namespace exmoe {

namespace {

constexpr int kClThreads = 512;
constexpr int kClWarps = kClThreads / 32;
constexpr int kClMaxUnits = 64;                      // (panel, K range) units per GEMM and CTA
constexpr int kClSmemLimit = 225 * 1024;           // dynamic; leaves room for the few static words

struct ClusterArgs {
    const uint8_t* slots;
    size_t slot_stride;
    size_t w13_bytes;
    const int32_t* ids;
    const int32_t* slot_of;                          // null: slot = expert id (C = E)
    const __nv_bfloat16* hidden;
    const float* topk_w;
    float* yk;                                       // [T*k, ks_d, H] unweighted partial down results per K range
    __nv_bfloat16* out;                              // [T, H]
    int* arrive;                                     // [T * CS] arrival counters (one per column slice), zero between calls
    int* status;
    int32_t* saved_ids;
    int E, k, H, I, n_pairs;
    int bpw_g, ks_g, bpw_d, ks_d;                    // blocks per K range / ranges, gate/up and down
    int ks_g_log2;
    int npp, npd;                                    // panel pairs (gate/up) and panels (down) per CTA
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
// relaxed: the only thing the other CTAs need from this one is its initialised mbarrier (published by
// fence.mbarrier_init); a releasing arrive would wait for every weight load in flight
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
// 16-byte store into another CTA's shared memory; completes 16 transaction bytes on that CTA's mbarrier
__device__ __forceinline__ void st_async16(uint32_t remote_addr, const uint4& v, uint32_t remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
    if (mbar_try_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned polls = 0;
    while (!mbar_try_cluster(bar, parity)) {
        if ((++polls & 15u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitBudget) {
                *abort_flag = 1;
                atomicExch(status, EXMOE_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
#ifdef EXMOE_CLUSTER_PROF
__device__ __forceinline__ unsigned long long gtime() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define CL_PROF(i) if (threadIdx.x == 0) prof_t[i] = gtime();
#define CL_WPROF(i) if ((threadIdx.x & 31) == 0) wprof[(threadIdx.x >> 5) * 8 + (i)] = gtime();
#else
#define CL_PROF(i)
#define CL_WPROF(i)
#endif

// NBG > 0: every warp holds its one gate/up unit (NBG blocks of gate and of up) in registers, loaded through the
//          load/store path, while the down slice comes through bulk copies: the two request paths run side by side
//          (bulk copies alone kept only ~25 KB per SM in flight, 2.6 TB/s over the chip).  Each warp is its own
//          pipeline: it stages the part of the hidden row its K range needs in a private piece of shared memory,
//          forms the block sums itself and starts on its weights as they arrive; the CTA first meets at the SwiGLU.
// NBG = 0: gate/up units through bulk copies into shared memory as well (any number of units per warp).
template <int NBG>
__global__ void __launch_bounds__(kClThreads, 1)
cluster_decode_kernel(ClusterArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
#ifdef EXMOE_CLUSTER_PROF
    unsigned long long prof_t[14] = {};
    __shared__ unsigned long long wprof[16 * 8];
    CL_PROF(0)
#endif
    // grid = (CS * ks_d, k, T): blockIdx.x = (K range of the down projection, rank in the cluster), pair p = t * k + j
    constexpr bool REGS = NBG > 0;
    constexpr int NBR = REGS ? NBG : 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q = lane >> 2, c = lane & 3;
    const int j = blockIdx.y, t = blockIdx.z, p = t * a.k + j;
    const uint32_t rank = cluster_ctarank(), CS = cluster_nctarank();
    const int rg = (int)(blockIdx.x / CS);
    const int KBg = a.H / kGroup, KBd = a.I / kGroup;
    const int Ug = a.npp << a.ks_g_log2, Ud = a.npd;
    const int Ugs = REGS ? 0 : Ug;                                               // gate/up units staged in shared memory
    const int Uds = REGS ? 0 : Ud;                                               // down units that arrive by bulk copy (mbarriers)
    const uint32_t gu_unit_bytes = 2u * a.bpw_g * kBlockBytes, dn_unit_bytes = (uint32_t)a.bpw_d * kBlockBytes;
    const int xs_bytes = REGS ? kClWarps * NBR * kGroup * 2 : a.H * 2;           // REGS: one K range of the row per warp

    uint64_t* bar_g = reinterpret_cast<uint64_t*>(smem);                         // [Ugs]
    uint64_t* bar_d = bar_g + Ugs;                                               // [Uds]
    uint64_t* bar_act = bar_d + Uds;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_act + 1);
    int* s_meta = const_cast<int*>(abort_flag) + 1;                              // [0] valid-id mask of the token, [1] last arriver
    float* s_rw = reinterpret_cast<float*>(s_meta + 2);                          // [32] routing weights of the token
    unsigned char* wgu = smem + (((size_t)(Ugs + Uds + 1) * 8 + 144 + 127) & ~(size_t)127);  // [Ugs][gate range | up range]
    unsigned char* wdn = wgu + (size_t)Ugs * gu_unit_bytes;                      // [Ud][range]
    unsigned char* xs = wdn + (size_t)Ud * dn_unit_bytes;                        // hidden row (or per-warp ranges of it)
    unsigned char* as = xs + xs_bytes;                                           // the range's activations, 128 * bpw_d BF16
    unsigned char* mine = as + (size_t)a.bpw_d * kGroup * 2;                     // this CTA's npp*16 activations
    float* adj_g = reinterpret_cast<float*>(mine + (size_t)a.npp * 32);          // [KBg]
    float* adj_d = adj_g + KBg;                                                  // [bpw_d]
    float* red_g = adj_d + a.bpw_d;                                              // [Ug][2][16]

    // Loads that do not depend on the ids go first: the hidden row (REGS: this warp's K range of it).
    const unsigned char* xrow_g = reinterpret_cast<const unsigned char*>(a.hidden + (size_t)t * a.H);
    const int x_chunks = a.H / 8;
    const int my_pp = warp >> a.ks_g_log2, my_ks = warp & ((1 << a.ks_g_log2) - 1);
    constexpr int XL = REGS ? (NBR * 16 + 31) / 32 : 1;                          // 16-byte chunks of the row per lane
    uint4 xpre[XL];
#pragma unroll
    for (int i = 0; i < XL; ++i) xpre[i] = make_uint4(0, 0, 0, 0);
    if (REGS) {
#pragma unroll
        for (int i = 0; i < XL; ++i)
            if (i * 32 + lane < NBR * 16) xpre[i] = ldg_early128(xrow_g + ((size_t)my_ks * NBR * 16 + i * 32 + lane) * 16);
    } else if (tid < x_chunks) {
        xpre[0] = ldg_early128(xrow_g + tid * 16);
    }
    const int id = a.ids[p];
    const bool id_ok = (unsigned)id < (unsigned)a.E;
    const int slot = id_ok ? (a.slot_of ? a.slot_of[id] : id) : 0;
    const uint8_t* wbase = a.slots + (size_t)slot * a.slot_stride;
    const size_t pp0 = (size_t)rg * a.bpw_d * (kGroup / kPanelRows) + (size_t)rank * a.npp;   // first panel pair of this CTA
    CL_PROF(1)
    // Thread u owns barrier u: it initialises it and, for a weight unit, requests the unit's bytes at once (bulk copy).
    if (tid <= Ugs + Uds) {
        mbar_init(bar_g + tid, 1);                                               // bar_g, bar_d and bar_act are contiguous
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (tid == Ugs + Uds) {
            *abort_flag = 0;
            mbar_expect_tx(bar_act, (uint32_t)a.bpw_d * kGroup * 2);             // CS parts of npp*32 bytes
        } else if (id_ok && tid < Ugs) {
            const int pp = tid >> a.ks_g_log2, ks = tid & ((1 << a.ks_g_log2) - 1);
            const size_t panel2 = 2 * (pp0 + pp);
            const uint8_t* src_g = wbase + ((panel2 + 0) * KBg + (size_t)ks * a.bpw_g) * kBlockBytes;
            const uint8_t* src_u = wbase + ((panel2 + 1) * KBg + (size_t)ks * a.bpw_g) * kBlockBytes;
            unsigned char* dst = wgu + (size_t)tid * gu_unit_bytes;
            mbar_expect_tx(bar_g + tid, gu_unit_bytes);
            bulk_g2s(dst, src_g, gu_unit_bytes / 2, bar_g + tid);
            bulk_g2s(dst + gu_unit_bytes / 2, src_u, gu_unit_bytes / 2, bar_g + tid);
        } else if (id_ok) {
            const int u = tid - Ugs;
            const uint8_t* src = wbase + a.w13_bytes + (((size_t)rank * a.npd + u) * KBd + (size_t)rg * a.bpw_d) * kBlockBytes;
            mbar_expect_tx(bar_d + u, dn_unit_bytes);
            bulk_g2s(wdn + (size_t)u * dn_unit_bytes, src, dn_unit_bytes, bar_d + u);
        }
    }

    if (warp == 1) {                                                             // which of the token's k ids are valid
        const bool v = lane < a.k && (unsigned)a.ids[t * a.k + lane] < (unsigned)a.E;
        const unsigned m = __ballot_sync(0xffffffffu, v);
        if (lane == 0) s_meta[0] = (int)m;
        if (lane < a.k) s_rw[lane] = a.topk_w[t * a.k + lane];
    }
    if ((blockIdx.x | blockIdx.y | blockIdx.z) == 0 && tid < a.n_pairs) {        // keep the ids (plan on request), flag bad ones
        const int v = a.ids[tid];
        a.saved_ids[tid] = v;
        if ((unsigned)v >= (unsigned)a.E) atomicExch(a.status, EXMOE_ERR_BAD_EXPERT_ID);
    }
    const int col0 = (int)rank * a.npd * kPanelRows, ncols = a.npd * kPanelRows;
    if (!id_ok) {
        // The pair contributes nothing (uniform over the cluster: none of its CTAs touches the cluster protocol).
        // A token without any valid id gets a zero row, written by the first cluster of its pair j = 0.
        __syncthreads();
        if (s_meta[0] == 0 && j == 0 && rg == 0)
            for (int col = tid; col < ncols; col += kClThreads) a.out[(size_t)t * a.H + col0 + col] = __float2bfloat16_rn(0.f);
        return;
    }
    CL_PROF(2)
    cluster_arrive();                                   // "my barriers exist"; waited for right before the exchange

    bool ok = true;
    if (REGS) {
        // ---- this warp's gate/up unit goes straight into registers, block by block, two blocks ahead of the arithmetic
        // (a warp that has issued everything first sits out the load queue's back-pressure with nothing to compute);
        // its part of the hidden row goes into its own piece of shared memory; adjv[b] = -136 * (block sum), formed as
        // the staging loops of the other decode kernels form it.  The warp's down units follow on the same path
        // (cp.async into shared memory: the warp that copies a unit consumes it).
        uint4 wreg[NBR][2][2];
        uint32_t sreg[NBR][2];
        float adjv[NBR];
        unsigned char* xw = xs + (size_t)warp * NBR * kGroup * 2;
        const bool has_unit = warp < Ug;
        const uint8_t* gu_base = wbase + (2 * (pp0 + my_pp) * KBg + (size_t)my_ks * NBR) * kBlockBytes;
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
            for (int u = warp; u < Ud; u += kClWarps) {
                const uint8_t* src = wbase + a.w13_bytes + (((size_t)rank * a.npd + u) * KBd + (size_t)rg * a.bpw_d) * kBlockBytes;
                unsigned char* dst = wdn + (size_t)u * dn_unit_bytes;
                for (uint32_t off = lane * 16; off < dn_unit_bytes; off += 32 * 16) cp_async16(dst + off, src + off);
            }
        };
#ifndef EXMOE_CLUSTER_AHEAD
#define EXMOE_CLUSTER_AHEAD 2
#endif
        constexpr int AHEAD = EXMOE_CLUSTER_AHEAD < NBR ? EXMOE_CLUSTER_AHEAD : NBR;    // blocks requested before the arithmetic starts
#pragma unroll
        for (int b = 0; b < AHEAD; ++b) issue_block(b);
        if (AHEAD == NBR) issue_down();
#pragma unroll
        for (int i = 0; i < XL; ++i) {
            const int ck = i * 32 + lane;
            if (ck < NBR * 16) *reinterpret_cast<uint4*>(xw + ck * 16) = xpre[i];
            float sx = sum8_bf16(xpre[i]);
#pragma unroll
            for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
            const float lo = __shfl_sync(0xffffffffu, sx, 0), hi = __shfl_sync(0xffffffffu, sx, 16);
            // __fmul_rn: the product is rounded on its own, as where the other kernels keep it in shared memory
            // (left to the compiler it would be contracted into the accumulator addition that uses it)
            if (2 * i < NBR) adjv[2 * i] = __fmul_rn(-136.f, lo);
            if (2 * i + 1 < NBR) adjv[2 * i + 1] = __fmul_rn(-136.f, hi);
        }
        __syncwarp();
        CL_WPROF(0)
        float tot[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
        for (int b = 0; b < NBR; ++b) {
            if (b + AHEAD < NBR) issue_block(b + AHEAD);
            if (AHEAD < NBR && b + AHEAD + 1 == NBR) issue_down();   // behind the last gate/up block
            if (b == 0) { CL_WPROF(1) }
            if (has_unit) chain_block_regs(wreg[b], sreg[b], adjv[b], b, xw, lane, tot);
        }
        CL_WPROF(2)
        if (has_unit && c == 0) {
            float* r = red_g + (size_t)warp * 32;
            r[q] = tot[0][0];
            r[q + 8] = tot[0][1];
            r[16 + q] = tot[1][0];
            r[16 + q + 8] = tot[1][1];
        }
    } else {
        // ---- stage the hidden row, adj_g[kb] = -136 * block sums
        for (int ck = tid; ck < x_chunks; ck += kClThreads) {
            const uint4 v = (ck < kClThreads) ? xpre[0] : *reinterpret_cast<const uint4*>(xrow_g + ck * 16);
            *reinterpret_cast<uint4*>(xs + ck * 16) = v;
        }
        __syncthreads();
        block_sums(xs, x_chunks, adj_g, warp, lane, kClThreads);
        __syncthreads();
        CL_PROF(3)
        // ---- gate/up: one (panel pair, K range) unit at a time per warp
        for (int u = warp; u < Ug; u += kClWarps) {
            const int ks = u & ((1 << a.ks_g_log2) - 1);
            ok = mbar_wait(bar_g + u, 0, abort_flag, a.status) && ok;
            const unsigned char* base = wgu + (size_t)u * gu_unit_bytes;
            const unsigned char* const w[2] = {base, base + gu_unit_bytes / 2};
            float tot[2][2];
            range_chain<2>(w, a.bpw_g, ks * a.bpw_g, xs, adj_g, lane, tot);
            if (c == 0) {
                float* r = red_g + (size_t)u * 32;
                r[q] = tot[0][0];
                r[q + 8] = tot[0][1];
                r[16 + q] = tot[1][0];
                r[16 + q + 8] = tot[1][1];
            }
        }
    }
    __syncthreads();
    CL_PROF(4)
#if EXMOE_CLUSTER_ABLATE == 1
    cp_async_wait_all();
    cluster_wait();
    return;                                             // timing only: through the gate/up arithmetic
#endif
    const unsigned valid_mask = (unsigned)s_meta[0];
    // K ranges added in ascending order, SwiGLU, one rounding to BF16
    for (int i = tid; i < a.npp * kPanelRows; i += kClThreads) {
        const int pp = i >> 4, r = i & 15;
        const float* base = red_g + ((size_t)pp << a.ks_g_log2) * 32;
        float g = base[r], u = base[16 + r];
        for (int s = 1; s < (1 << a.ks_g_log2); ++s) {
            g += base[s * 32 + r];
            u += base[s * 32 + 16 + r];
        }
        reinterpret_cast<__nv_bfloat16*>(mine)[i] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * u);
    }
    __syncthreads();

    // ---- exchange: this CTA's activations to every CTA of the cluster (its own included)
    cluster_wait();
    {
        const int chunks = a.npp * 2;                   // 16-byte chunks of this CTA's part
        const uint32_t as_addr = smem_u32(as) + rank * (uint32_t)(a.npp * 32), bar_addr = smem_u32(bar_act);
        for (int i = tid; i < (int)CS * chunks; i += kClThreads) {
            const uint32_t dst = (uint32_t)(i / chunks), ch = (uint32_t)(i - (int)dst * chunks);
            const uint4 v = *reinterpret_cast<const uint4*>(mine + ch * 16);
            st_async16(map_to_rank(as_addr + ch * 16, dst), v, map_to_rank(bar_addr, dst));
        }
    }
    CL_PROF(5)
    ok = mbar_wait_cluster(bar_act, 0, abort_flag, a.status) && ok;
    CL_PROF(6)
#if EXMOE_CLUSTER_ABLATE == 2
    cp_async_wait_all();
    return;                                             // timing only: through the exchange
#endif
    block_sums(as, a.bpw_d * (kGroup / 8), adj_d, warp, lane, kClThreads);
    __syncthreads();
#ifdef EXMOE_CLUSTER_PROF
    if (REGS) { CL_PROF(3) }
#endif

    // ---- this K range's partial down projection of this CTA's output rows (unweighted)
    float* ypart = a.yk + ((size_t)p * a.ks_d + rg) * a.H + col0;
    CL_WPROF(3)
    if (REGS) {
        cp_async_wait_all();                            // this lane's pieces of the warp's down units ...
        __syncwarp();                                   // ... and the other lanes'
    }
    CL_WPROF(4)
    for (int u = warp; u < Ud; u += 2 * kClWarps) {     // two units at a time: independent accumulator chains, shared fragments
        const int u2 = u + kClWarps;
        if (!REGS) {
            ok = mbar_wait(bar_d + u, 0, abort_flag, a.status) && ok;
            if (u2 < Ud) ok = mbar_wait(bar_d + u2, 0, abort_flag, a.status) && ok;
        }
        if (u2 < Ud) {
            const unsigned char* const w[2] = {wdn + (size_t)u * dn_unit_bytes, wdn + (size_t)u2 * dn_unit_bytes};
            float tot[2][2];
            if (a.bpw_d == 2) unit_chains<2, 2>(w, as, adj_d, lane, tot);       // the usual range of two blocks, unrolled
            else if (a.bpw_d == 1) unit_chains<2, 1>(w, as, adj_d, lane, tot);
            else range_chain<2>(w, a.bpw_d, 0, as, adj_d, lane, tot);
            if (c == 0 && ok) {
                ypart[u * kPanelRows + q] = tot[0][0];
                ypart[u * kPanelRows + q + 8] = tot[0][1];
                ypart[u2 * kPanelRows + q] = tot[1][0];
                ypart[u2 * kPanelRows + q + 8] = tot[1][1];
            }
        } else {
            const unsigned char* const w[1] = {wdn + (size_t)u * dn_unit_bytes};
            float tot[1][2];
            range_chain<1>(w, a.bpw_d, 0, as, adj_d, lane, tot);
            if (c == 0 && ok) {
                ypart[u * kPanelRows + q] = tot[0][0];
                ypart[u * kPanelRows + q + 8] = tot[0][1];
            }
        }
    }
    CL_PROF(10)
    CL_WPROF(5)
    ok = __syncthreads_and(ok ? 1 : 0) != 0;
    CL_PROF(7)
#if EXMOE_CLUSTER_ABLATE == 3
    return;                                             // timing only: through the down projection
#endif
    if (!ok) {
        // a wait expired (status raised): write nothing; give copies that may still be in flight a bounded time to land
        if (tid == 0) {
            const long long t0 = clock64();
            for (int u = 0; u < Ugs + Uds; ++u)
                while (!mbar_try(bar_g + u, 0) && clock64() - t0 < kWaitBudget) {}
        }
        return;
    }

    // ---- Eq. 2's sum over the selected experts.  Every (valid pair, K range) cluster reports once per column slice;
    // the CTA whose report completes a slice forms each pair's result (K ranges in ascending order, x routing weight)
    // and adds the k pair rows in the fixed order j = 0..k-1.
    if (tid == 0) {
        // one acquire-release atomic at device scope: it publishes the CTA's partial rows (ordered before it by the
        // barrier above) and, for the last arriver, makes the other clusters' rows visible to the reads below
        const int need = __popc(valid_mask) * a.ks_d;
        int* ctr = a.arrive + t * (int)CS + (int)rank;
        int old;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(ctr) : "memory");
        if (old == need - 1) *ctr = 0;                  // self-cleaning for the next call
        s_meta[1] = (old == need - 1);
    }
    __syncthreads();
#if EXMOE_CLUSTER_ABLATE == 4
    return;                                             // timing only: everything but the last arriver's sum
#endif
    if (s_meta[1]) {
        CL_PROF(9)
        // (pair, four columns) items: a pair's K ranges are added in ascending order and weighted as they are loaded
        // (independent 128-bit loads, four ranges in flight per item), then the k pair rows are added in order
        const int vps = ncols / 4;                                               // float4 per row of the slice
        float4* ys = reinterpret_cast<float4*>(wgu);                             // [k][vps]
        const float* ybase = a.yk + (size_t)t * a.k * a.ks_d * a.H + col0;
        const size_t row4 = (size_t)a.H / 4;
#pragma unroll 2
        for (int i = tid; i < a.k * vps; i += kClThreads) {
            const int jj = i / vps, v = i - jj * vps;
            const float4* src = reinterpret_cast<const float4*>(ybase + (size_t)jj * a.ks_d * a.H) + v;
            float4 res = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r0 = 0; r0 < a.ks_d; r0 += 4) {
                float4 x[4];
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    x[r] = (r0 + r < a.ks_d) ? __ldcg(src + (size_t)(r0 + r) * row4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (r0 + r >= a.ks_d) break;
                    if (r0 + r == 0) { res = x[0]; continue; }
                    res.x = __fadd_rn(res.x, x[r].x); res.y = __fadd_rn(res.y, x[r].y);
                    res.z = __fadd_rn(res.z, x[r].z); res.w = __fadd_rn(res.w, x[r].w);
                }
            }
            const float rw = s_rw[jj];                  // the product is rounded on its own, as in the other kernels
            ys[i] = make_float4(__fmul_rn(rw, res.x), __fmul_rn(rw, res.y), __fmul_rn(rw, res.z), __fmul_rn(rw, res.w));
        }
        __syncthreads();
        CL_PROF(11)
        for (int col = tid; col < ncols; col += kClThreads) {
            float sum = 0.f;
            for (int jj = 0; jj < a.k; ++jj)
                if ((valid_mask >> jj) & 1u) sum = __fadd_rn(sum, reinterpret_cast<const float*>(ys)[(size_t)jj * ncols + col]);
            a.out[(size_t)t * a.H + col0 + col] = __float2bfloat16_rn(sum);
        }
    }
#ifdef EXMOE_CLUSTER_PROF
    CL_PROF(8)
    if (tid == 0) {
        { const long long c0 = clock64(); while (clock64() - c0 < 100000) {} }   // debug build only: print after everybody has finished
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        printf("CL x=%d j=%d t=%d sm=%u last=%d t0=%llu ids=%llu issue=%llu staged=%llu gu=%llu sent=%llu act=%llu down=%llu end=%llu c9=%llu c10=%llu c11=%llu\n",
               (int)blockIdx.x, j, t, smid, s_meta[1], prof_t[0], prof_t[1] - prof_t[0], prof_t[2] - prof_t[0],
               prof_t[3] - prof_t[0], prof_t[4] - prof_t[0], prof_t[5] - prof_t[0], prof_t[6] - prof_t[0], prof_t[7] - prof_t[0],
               prof_t[8] - prof_t[0], prof_t[9] - prof_t[0], prof_t[10] - prof_t[0], prof_t[11] - prof_t[0]);
        if (blockIdx.x == 5 && j == 3)
            for (int w = 0; w < 16; ++w)
                printf("W %d issued=%llu chain0=%llu chain1=%llu dwait0=%llu dwait1=%llu ddone=%llu\n", w, wprof[w * 8] - prof_t[0],
                       wprof[w * 8 + 1] - prof_t[0], wprof[w * 8 + 2] - prof_t[0], wprof[w * 8 + 3] - prof_t[0],
                       wprof[w * 8 + 4] - prof_t[0], wprof[w * 8 + 5] - prof_t[0]);
    }
#endif
}

struct ClusterCfg {
    int cs, npp, npd, bpw_g, ks_g, bpw_d, ks_d, nbg;
    size_t smem;
};

size_t cluster_smem_bytes(int H, const ClusterCfg& c) {
    const int Ug = c.npp * c.ks_g, Ud = c.npd, Ugs = c.nbg ? 0 : Ug, Uds = c.nbg ? 0 : Ud;
    const size_t xs_bytes = c.nbg ? (size_t)kClWarps * c.nbg * kGroup * 2 : (size_t)H * 2;
    return (((size_t)(Ugs + Uds + 1) * 8 + 144 + 127) & ~(size_t)127) + (size_t)Ugs * 2 * c.bpw_g * kBlockBytes +
           (size_t)Ud * c.bpw_d * kBlockBytes + xs_bytes + (size_t)c.bpw_d * kGroup * 2 + (size_t)c.npp * 32 +
           (size_t)(H / kGroup + c.bpw_d) * 4 + (size_t)Ug * 32 * 4 + 128;
}

using ClusterKernel = void (*)(ClusterArgs);
ClusterKernel cluster_kernel(int nbg) {
    return nbg == 4 ? cluster_decode_kernel<4> : nbg == 2 ? cluster_decode_kernel<2> : nbg == 1 ? cluster_decode_kernel<1>
                                                                                             : cluster_decode_kernel<0>;
}

}  // namespace

// The K ranges of the other decode kernels (decode.cu: pick_cfg), which this kernel replays for identical rounding.
void decode_k_split(int K, int rows, bool down, int* ks, int* bpw);

// 0 = this device cannot co-schedule a cluster of `cs` CTAs of this kernel with `smem` bytes each
static int max_active_clusters(ClusterKernel kern, int cs, size_t smem) {
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(cs, 1, 1);
    lc.blockDim = dim3(kClThreads);
    lc.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &lc) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

static std::atomic<int> g_force_cs{0};
void cluster_force_size(int cs) { g_force_cs.store(cs); }
int cluster_forced_size() { return g_force_cs.load(); }

size_t cluster_partial_floats(int H, int I) {
    int ks = 1, bpw = 1;
    decode_k_split(I, H, true, &ks, &bpw);
    return (size_t)kSmallMaxPairs * ks * H;
}

// Launches the one-kernel layer when the shape fits a small cluster's shared memory; false = not taken (nothing queued).
bool launch_cluster_decode(const GemmArgs& g, const SmallWave& w, cudaStream_t st) {
#ifdef EXMOE_NO_CLUSTER_DECODE
    return false;
#endif
    const int H = g.H, I = g.I, k = g.top_k;
    const int forced = g_force_cs.load();
    // larger tiny batches run their clusters in several rounds and measured slower than the per-pair kernels; the test
    // hook still sends them here
    if (k > 32 || w.n_pairs > (forced ? kSmallMaxPairs : kClusterMaxPairs) || w.n_pairs % k || !w.yk || !w.arrive) return false;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    ClusterCfg cfg{};
    decode_k_split(H, I, false, &cfg.ks_g, &cfg.bpw_g);
    decode_k_split(I, H, true, &cfg.ks_d, &cfg.bpw_d);
    int ks_g_log2 = 0;
    while ((1 << ks_g_log2) < cfg.ks_g) ++ks_g_log2;
    if ((1 << ks_g_log2) != cfg.ks_g) return false;
    // occupancy answers are cached per (device, cluster size, shape)
    struct Seen { int H, I, cs; bool fits; };
    static Seen seen[64][8];
    static int n_seen[64] = {};
    static SmemOnce smem_once[4];
    bool found = false;
    const int range_pp = cfg.bpw_d * (kGroup / kPanelRows);         // panel pairs whose activations one K range needs
    // the smallest cluster whose CTAs fit their slices (the most bytes in flight per SM); portable sizes only
    for (int cs = 1; cs <= 8 && !found; cs <<= 1) {
        if (forced && cs != forced) continue;
        if (range_pp % cs || H % (kPanelRows * cs)) continue;
        cfg.cs = cs;
        cfg.npp = range_pp / cs;
        cfg.npd = H / (kPanelRows * cs);
        if (cfg.npp * cfg.ks_g > kClMaxUnits || cfg.npd > kClMaxUnits) continue;
        // one gate/up unit per warp and 1, 2 or 4 blocks per unit: the unit lives in registers
        cfg.nbg = (cfg.npp * cfg.ks_g <= kClWarps && (cfg.bpw_g == 1 || cfg.bpw_g == 2 || cfg.bpw_g == 4)) ? cfg.bpw_g : 0;
#ifdef EXMOE_CLUSTER_FORCE_BULK
        cfg.nbg = 0;
#endif
        cfg.smem = cluster_smem_bytes(H, cfg);
        if (cfg.smem > (size_t)kClSmemLimit) continue;
        // the final sum stages k x (slice columns) floats where the weights were
        const size_t wbytes = (size_t)(cfg.nbg ? 0 : cfg.npp * cfg.ks_g) * 2 * cfg.bpw_g * kBlockBytes + (size_t)cfg.npd * cfg.bpw_d * kBlockBytes;
        if ((size_t)k * cfg.npd * kPanelRows * 4 > wbytes) continue;
        ClusterKernel kern = cluster_kernel(cfg.nbg);
        if (!allow_smem(kern, kClSmemLimit, smem_once[cfg.nbg == 4 ? 3 : cfg.nbg])) {
            cudaGetLastError();
            return false;
        }
        bool known = false, fits = false;
        for (int i = 0; i < n_seen[dev]; ++i)
            if (seen[dev][i].H == H && seen[dev][i].I == I && seen[dev][i].cs == cs) { known = true; fits = seen[dev][i].fits; }
        if (!known) {
            fits = max_active_clusters(kern, cs, cfg.smem) >= 1;
            if (n_seen[dev] < 8) seen[dev][n_seen[dev]++] = Seen{H, I, cs, fits};
        }
        found = fits;
    }
    if (!found) return false;

    ClusterArgs a{};
    a.slots = g.slots;
    a.slot_stride = g.slot_stride;
    a.w13_bytes = matrix_bytes(2 * I, H);
    a.ids = w.ids;
    a.slot_of = w.slot_of;
    a.hidden = w.hidden;
    a.topk_w = w.topk_w;
    a.yk = w.yk;
    a.out = w.out;
    a.arrive = w.arrive;
    a.status = w.status;
    a.saved_ids = w.saved_ids;
    a.E = w.E;
    a.k = k;
    a.H = H;
    a.I = I;
    a.n_pairs = w.n_pairs;
    a.bpw_g = cfg.bpw_g; a.ks_g = cfg.ks_g; a.bpw_d = cfg.bpw_d; a.ks_d = cfg.ks_d;
    a.ks_g_log2 = ks_g_log2;
    a.npp = cfg.npp; a.npd = cfg.npd;

    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(cfg.cs * cfg.ks_d, k, w.n_pairs / k);
    lc.blockDim = dim3(kClThreads);
    lc.dynamicSmemBytes = cfg.smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cfg.cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, cluster_kernel(cfg.nbg), a) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    count_launch();
    return true;
}

}  // namespace exmoe
