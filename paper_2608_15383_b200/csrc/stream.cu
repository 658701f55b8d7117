// Streaming grouped W4A16 kernels for the middle regime (a few to a few dozen rows per expert): the two
// grouped expert GEMMs of a wave (Section 3.4, Eq. 2) as HBM-bound streams over the packed expert bytes,
// with the memory system decoupled from the arithmetic.
//
// The work of a wave is cut into units: (active group = expert, pass over up to 8 or 16 of the group's rows,
// tile of PP panels; gate/up: PP gate+up panel pairs).  A tile is ONE contiguous range of the packed
// expert image.  Units are ordered group-major, then pass, then tile, and every persistent CTA (one per
// SM) takes an equal contiguous share, so that the load is balanced by arithmetic, not by expert, and a
// CTA's consecutive units share their activation rows.  A group with more rows than one pass holds
// re-reads its tiles once per pass (they come from L2).  Roles by warp:
//   warps 0-15  two consumer groups of eight warps that take alternate units: read the tile's packed bytes
//               from shared memory (the image is already in m16n8k16 fragment order), dequantise in
//               registers (shift + lop3), mma.sync against the group's activation rows, scale per 128-wide
//               block in binary32; the K-split partials cross shared memory once and every warp finishes
//               a slice of the tile (fixed summation order; SwiGLU or routing weight; store).
//   warp 16     weight producer: one cp.async.bulk per unit into a ring of stages, completion counted in
//               bytes on the stage's mbarrier; runs as many stages ahead as the ring is deep.
//   warp 17     activation producer: one cp.async.bulk per activation row (gathered through the plan's
//               permutation for gate/up) into a row buffer (two of them where shared memory allows).
// The down kernel is a programmatic dependent of the gate/up kernel: its weight ring fills while the
// gate/up kernel drains; only its activation producer waits for the dependency.
// Every mbarrier wait is bounded: on expiry the CTA raises EXMOE_ERR_TIMEOUT, all roles leave their
// loops and the producers wait (bounded) for their copies in flight before the CTA exits.
#include "common.cuh"
#include "frag.cuh"
#include "mbar.cuh"
#ifdef EXMOE_STREAM_PROF
#include <cstdio>
#define SPROF(...) __VA_ARGS__
#else
#define SPROF(...)
#endif

namespace exmoe {

namespace {

constexpr int kGroupWarps = 8;                       // warps of one consumer group
constexpr int kGroupThreads = 32 * kGroupWarps;
constexpr int kGroups = 2;                           // consumer groups, alternate units
constexpr int kConsumerWarps = kGroups * kGroupWarps;
constexpr int kStreamThreads = 32 * (kConsumerWarps + 2);
constexpr int kMaxStages = 8;
constexpr size_t kSmemLimit = 227 * 1024;
constexpr int kScanChunks = 4;                       // chunks of 32 groups whose plan entries the scan keeps in registers
constexpr int kMetaGroups = 64;                      // most groups one CTA's share of the units can touch (see stream_geometry)

// one lane waits, the whole warp learns the outcome (the producers' control flow stays warp-uniform)
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// untiled bulk copy global -> shared (both 16-byte aligned, size a multiple of 16), no multicast
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void group_sync(int grp) {              // named barrier of one consumer group
    asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "n"(kGroupThreads) : "memory");
}

struct StreamGeom {
    int PP, KS, NMW, tiles, n_stages, n_xbuf;
    uint32_t stage_bytes, x_stride;
    size_t off_x, off_part, off_adj, off_bar, total;
};

constexpr size_t kBarBytes = (2 * kMaxStages + 4) * 8 + 64;          // mbarriers, abort flag, unit range
constexpr size_t kCtrlBytes = kBarBytes + (size_t)kMetaGroups * 16;  // + plan entries of the CTA's groups

#ifndef EXMOE_STREAM_PP
#define EXMOE_STREAM_PP 0                                              // 0: choose; 1/2/4/8: force where feasible (timing experiments)
#endif

// Tile shape and shared-memory budget for one matrix kind.  The eight warps of a consumer group are
// PP panels x (gate | up, when a warp holds one of the two: NMW = 1) x KS ranges of K.
// Preference: a ring of at least four stages, then two activation buffers over one, then the larger tile.
__host__ bool stream_geometry(int K, int NR, int NM, int NCH, StreamGeom* out) {
    const int KB = K / kGroup, R = 8 * NCH;
    const size_t x_stride = (size_t)K * 2 + 64;
    long best = -1;
    for (int NX = 2; NX >= 1; --NX)
        for (int PP = 8; PP >= 1; PP >>= 1) {
            const int NMW = (NM == 2 && PP == 8) ? 2 : 1;              // both matrices in one warp only when there is no room to split
            const int KS = 8 / (PP * (NM / NMW));
            if (KS < 1 || KB % KS || NR % (kPanelRows * PP)) continue;
            if (EXMOE_STREAM_PP && PP != EXMOE_STREAM_PP) continue;
            const size_t stage = (size_t)NM * PP * KB * kBlockBytes;
            if (stage > 96 * 1024) continue;
            const size_t xs = (size_t)NX * R * x_stride;
            const bool exchange = !(KS == 1 && NMW == NM);             // partials cross shared memory
            const size_t part = exchange ? (size_t)kGroups * 2 * kGroupWarps * NMW * NCH * 512 : 0;
            const size_t adj = (size_t)kGroups * NX * KB * R * 4;
            const size_t fixed = xs + part + adj + kCtrlBytes + 192;
            if (fixed + 2 * stage > kSmemLimit) continue;
            int S = (int)((kSmemLimit - fixed) / stage);
            if (S > kMaxStages) S = kMaxStages;
            const long score = (S >= 4 ? 2 : S == 3 ? 1 : 0) * 1000 + NX * 100 + PP;
            if (score <= best) continue;
            best = score;
            StreamGeom g{};
            g.PP = PP; g.KS = KS; g.NMW = NMW; g.tiles = NR / (kPanelRows * PP); g.n_stages = S; g.n_xbuf = NX;
            g.stage_bytes = (uint32_t)stage; g.x_stride = (uint32_t)x_stride;
            g.off_x = (size_t)S * stage;
            g.off_part = g.off_x + xs;
            g.off_adj = g.off_part + part;
            g.off_bar = (g.off_adj + adj + 63) & ~(size_t)63;
            g.total = g.off_bar + kCtrlBytes;
            *out = g;
        }
    return best >= 0;
}

struct StreamArgs {
    GemmArgs a;
    const __nv_bfloat16* x_src;     // gate/up: hidden [T, H]; down: activations [pairs, I] in grouped row order
    __nv_bfloat16* act_out;         // gate/up result
    const float* topk_w;
    float* y_out;                   // down result x routing weight, [pairs, H] in pair order
    int* status;
    int PP, KS, n_stages, n_xbuf;
    uint32_t stage_bytes, x_stride;
    uint32_t off_x, off_part, off_adj, off_bar;
};

// position of a unit inside the CTA's share: index into the cached plan entries, pass, tile
struct Cursor {
    int gi, pass, tile;
    __device__ __forceinline__ void advance(int tiles, int passes) {
        if (++tile == tiles) {
            tile = 0;
            if (++pass == passes) {
                pass = 0;
                ++gi;
            }
        }
    }
};

// NMW: matrices held by one warp (2 = gate and up of the same panel; 1 = one matrix, gate/up split over warps)
// KBc, PPc, KSc: blocks along K, panels per tile and K ranges per panel as COMPILE-TIME constants (0 = taken from the
// arguments).  With run-time values about a third of the executed instructions were address arithmetic, predicates and
// loop control around the conversion and the MMAs; the shapes that matter (OLMoE's two matrices) get their own
// instantiations with the block loop unrolled and every stride a literal, all others run the generic one.
template <int NCH, bool GATEUP, int NMW, int KBc = 0, int PPc = 0, int KSc = 0>
__global__ void __launch_bounds__(kStreamThreads, 1)
stream_gemm_kernel(const StreamArgs p) {
    constexpr int NM = GATEUP ? 2 : 1;                                // matrices per tile
    constexpr int MS = NM / NMW;                                      // warps a panel's matrices are split over
    constexpr int R = 8 * NCH;
    constexpr int CHN = (NMW * NCH >= 2) ? 1 : 2;                          // accumulator chains per (matrix, chunk): two independent MMA chains per warp at least
    extern __shared__ __align__(128) unsigned char smem[];
    const GemmArgs& a = p.a;
    constexpr bool FIXED = KBc > 0;
    constexpr int BPWc = KSc > 0 ? KBc / (KSc > 0 ? KSc : 1) : 0;     // blocks per K range when the geometry is fixed
    const int NR = GATEUP ? a.I : a.H;
    const int KB = FIXED ? KBc : (GATEUP ? a.H : a.I) / kGroup, K = KB * kGroup;
    const int PP = FIXED ? PPc : p.PP, KS = FIXED ? KSc : p.KS, bpw = KB / KS;
    const uint32_t x_stride = FIXED ? (uint32_t)(KBc * kGroup * 2 + 64) : p.x_stride;
    const uint32_t stage_bytes = FIXED ? (uint32_t)((GATEUP ? 2 : 1) * PPc * KBc * kBlockBytes) : p.stage_bytes;
    const int tiles = NR / (kPanelRows * PP);
    const int S = p.n_stages, NX = p.n_xbuf;
    unsigned char* wst = smem;
    unsigned char* xs = smem + p.off_x;
    float* part = reinterpret_cast<float*>(smem + p.off_part);
    float* adj = reinterpret_cast<float*>(smem + p.off_adj);
    uint64_t* w_full = reinterpret_cast<uint64_t*>(smem + p.off_bar);
    uint64_t* w_empty = w_full + kMaxStages;
    uint64_t* x_full = w_empty + kMaxStages;
    uint64_t* x_empty = x_full + 2;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(x_empty + 2);
    int* s_range = const_cast<int*>(abort_flag) + 4;                   // [0] first unit, [1] end
    const int4* meta = reinterpret_cast<const int4*>(smem + p.off_bar + kBarBytes);   // (key, rows, first row, first unit)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 32) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&w_full[s], 1);
            mbar_init(&w_empty[s], kConsumerWarps);                    // both groups: see the consumer loop
        }
        for (int b = 0; b < NX; ++b) {
            mbar_init(&x_full[b], 1);
            mbar_init(&x_empty[b], kConsumerWarps);                    // both groups
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
#ifndef EXMOE_STREAM_NO_ENTRY_PDL
    // The gate/up kernel is itself launched as a programmatic dependent (of the grouping kernel when that runs
    // just before it): its CTAs are placed and their barriers initialised while the plan is still being
    // written; the plan is read only after this wait.
    if (GATEUP) grid_dependency_wait();
#endif
    if (warp == 0) {
        // This CTA's share of the wave's units, and the plan entries of the groups it touches (usually one or
        // two).  The plan entries of up to 32 * kScanChunks active groups are fetched in one go and kept in
        // registers for both steps (count the units; find the overlapping groups); beyond that they are re-read.
        // With every expert resident the keys are the expert ids and the wave is the whole call: counts and offsets are
        // then read by key at once (empty keys are empty groups), one round trip to L2 instead of three dependent ones
        // (wave_start, then group_keys, then counts / offsets) before the first weight copy can be issued.
        const bool direct = a.direct_keys > 0 && a.direct_keys <= 32 * kScanChunks;
        const int g0 = direct ? 0 : a.wave_start[0], n_groups = direct ? a.direct_keys : a.wave_start[1] - g0;
        int rkey[kScanChunks], rrows[kScanChunks], rrow0[kScanChunks];
#pragma unroll
        for (int j = 0; j < kScanChunks; ++j) {
            rkey[j] = 0;
            if (32 * j + lane < n_groups) rkey[j] = direct ? 32 * j + lane : a.group_keys[g0 + 32 * j + lane];
        }
#pragma unroll
        for (int j = 0; j < kScanChunks; ++j) {
            rrows[j] = rrow0[j] = 0;
            if (32 * j + lane < n_groups) {
                rrows[j] = a.counts[rkey[j]];
                rrow0[j] = a.offsets[rkey[j]];
            }
        }
        // group filter (miss fetch overlapped with compute): a launch takes only the groups whose expert was resident
        // (1) or only those that were fetched for this wave (2); the others count as empty
        const int filter = a.key_miss ? a.group_filter : 0;
#pragma unroll
        for (int j = 0; j < kScanChunks; ++j)
            if (filter && 32 * j + lane < n_groups && (a.key_miss[rkey[j]] != 0) != (filter == 2)) rrows[j] = 0;
        auto entry = [&](int chunk, int& key, int& rows, int& row0) {
            key = rows = row0 = 0;
            bool have = false;
#pragma unroll
            for (int j = 0; j < kScanChunks; ++j)
                if (chunk == j) {
                    key = rkey[j];
                    rows = rrows[j];
                    row0 = rrow0[j];
                    have = true;
                }
            if (!have && 32 * chunk + lane < n_groups) {
                key = a.group_keys[g0 + 32 * chunk + lane];
                rows = a.counts[key];
                row0 = a.offsets[key];
                if (filter && (a.key_miss[key] != 0) != (filter == 2)) rows = 0;
            }
        };
        int total = 0;
        for (int chunk = 0; 32 * chunk < n_groups; ++chunk) {
            int key, rows, row0;
            entry(chunk, key, rows, row0);
            int passes = (rows + R - 1) / R;
#pragma unroll
            for (int m = 16; m >= 1; m >>= 1) passes += __shfl_xor_sync(0xffffffffu, passes, m);
            total += passes;
        }
        const long long U = (long long)total * tiles;
        int u0 = (int)(U * blockIdx.x / gridDim.x), u1 = (int)(U * (blockIdx.x + 1) / gridDim.x);
        int run = 0, found = 0;
        int4* meta_w = const_cast<int4*>(meta);
        for (int chunk = 0; 32 * chunk < n_groups && u0 < u1; ++chunk) {
            int key, rows, row0;
            entry(chunk, key, rows, row0);
            const int passes = (rows + R - 1) / R;
            int incl = passes;
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, m);
                if (lane >= m) incl += v;
            }
            const int ustart = (run + incl - passes) * tiles, uend = ustart + passes * tiles;
            const bool overlap = passes > 0 && ustart < u1 && uend > u0;
            const unsigned ballot = __ballot_sync(0xffffffffu, overlap);
            if (overlap) {
                const int idx = found + __popc(ballot & ((1u << lane) - 1u));
                if (idx < kMetaGroups) meta_w[idx] = make_int4(key % a.num_slots, rows, row0, ustart);   // .x = slot of the group
            }
            found += __popc(ballot);
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (found > kMetaGroups) {                     // cannot happen for the sizes this path is chosen for; never index past the table
            if (lane == 0) atomicExch(p.status, EXMOE_ERR_STATE);
            u1 = u0;
        }
        if (lane == 0) {
            s_range[0] = u0;
            s_range[1] = u1;
        }
    }
    __syncthreads();
    grid_launch_dependents();                          // gate/up: the down kernel may start filling its weight ring; down: the
                                                       // combine kernel may be placed (it waits for this grid before it reads)
    const int u0 = s_range[0], u1 = s_range[1];
    const size_t mat_off = GATEUP ? 0 : matrix_bytes(2 * a.I, a.H);
    Cursor cur{0, 0, 0};
    if (u0 < u1) {
        const int off = u0 - meta[0].w;
        cur.pass = off / tiles;
        cur.tile = off % tiles;
    }

    if (warp == kConsumerWarps) {
        // ---------------------------------------------------------------- weight producer
        // ring position and phase are carried along: no division in any per-unit path of this kernel (a runtime
        // integer division costs some 25 instructions, several of them on the quarter-rate conversion pipe)
        int n = 0, s = 0;
        uint32_t ph = 1;                               // parity of the stage's previous phase
        for (int u = u0; u < u1; ++u, ++n) {
            if (n >= S && !warp_wait(&w_empty[s], ph, abort_flag, p.status)) break;
            const int4 gm = meta[cur.gi];
            if (lane == 0) {
                const uint8_t* src = a.slots + (size_t)gm.x * a.slot_stride + mat_off + (size_t)cur.tile * stage_bytes;
                mbar_expect_tx(&w_full[s], stage_bytes);
                bulk_load(wst + (size_t)s * stage_bytes, src, stage_bytes, &w_full[s]);
            }
            __syncwarp();
            cur.advance(tiles, (gm.y + R - 1) / R);
            if (++s == S) {
                s = 0;
                ph ^= 1u;
            }
        }
        if (*abort_flag && lane == 0) {                // copies in flight land before the shared memory is given up
            for (int j = (n > S ? n - S : 0); j < n; ++j) {
                const long long t0 = clock64();
                while (!mbar_try(&w_full[j % S], (j / S) & 1) && clock64() - t0 < kWaitBudget) {}
            }
        }
    } else if (warp == kConsumerWarps + 1) {
        // ---------------------------------------------------------------- activation producer
        if (!GATEUP) grid_dependency_wait();           // the gate/up kernel's activations are complete and visible
        int n = 0, b = 0;
        uint32_t ph = 1;
        for (int u = u0; u < u1; ++u) {
            const int4 gm = meta[cur.gi];
            if (u == u0 || cur.tile == 0) {            // first unit of a (group, pass): stage its rows
                if (n >= NX && !warp_wait(&x_empty[b], ph, abort_flag, p.status)) break;
                const int pass0 = cur.pass * R;
                const int rows_here = min(R, gm.y - pass0);
                if (lane == 0) mbar_expect_tx(&x_full[b], (uint32_t)rows_here * K * 2);
                __syncwarp();
                if (lane < rows_here) {
                    const size_t src_row = GATEUP ? (size_t)(a.perm[gm.z + pass0 + lane] / a.top_k)
                                                  : (size_t)(gm.z + pass0 + lane);
                    bulk_load(xs + ((size_t)b * R + lane) * x_stride, p.x_src + src_row * K, (uint32_t)K * 2, &x_full[b]);
                }
                __syncwarp();
                ++n;
                if (++b == NX) {
                    b = 0;
                    ph ^= 1u;
                }
            }
            cur.advance(tiles, (gm.y + R - 1) / R);
        }
        if (*abort_flag && lane == 0) {
            for (int j = (n > NX ? n - NX : 0); j < n; ++j) {
                const long long t0 = clock64();
                while (!mbar_try(&x_full[j % NX], (j / NX) & 1) && clock64() - t0 < kWaitBudget) {}
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers
        const int grp = warp / kGroupWarps, cw = warp % kGroupWarps;
        const int q = lane >> 2, c = lane & 3;
        const int ks = cw % KS, mw = (cw / KS) % MS, pp = cw / (KS * MS);    // K range, matrix (when split), panel
        const bool exchange = !(KS == 1 && MS == 1);
        // partials of one unit: [pp][matrix][ks][ch][i][lane], one buffer per group and unit parity
        const int part_words = kGroupWarps * NMW * NCH * 128;
        float* adjg = adj + (size_t)grp * NX * KB * R;
        int mine_cnt = 0;
        int s = -1, xb = -1;                           // weight stage and row buffer of the current unit
        uint32_t w_ph = 1, x_ph = 1;                   // their barrier parities (flipped when the index wraps to 0)
        // Both groups walk ALL units in order and observe every phase of every full barrier, also for units and
        // rows the other group computes on, and release each stage only then: a parity wait is only valid for a
        // waiter that is at most one phase behind.
        // A failed (expired or aborted) wait never changes the control flow: the named barriers below need all
        // eight warps of the group, so the thread runs on over whatever the buffers hold, stores nothing, and
        // every later wait returns at once because the abort flag is up.
        bool ok = true;
        SPROF(long long t_x = 0, t_w = 0, t_mma = 0, t_ep = 0, t_other = 0, t_begin = clock64(); int n_mine = 0;)
        for (int u = u0, n = 0; u < u1; ++u, ++n) {
            SPROF(long long c0 = clock64();)
            const int4 gm = meta[cur.gi];
            const int m_rows = gm.y, row0 = gm.z, tile = cur.tile, pass0 = cur.pass * R;
            const bool fresh = (u == u0 || tile == 0);
            const bool x_done = (u + 1 == u1 || tile == tiles - 1);
            cur.advance(tiles, (m_rows + R - 1) / R);
            if (fresh && ++xb == NX) xb = 0;
            if (fresh && xb == 0) x_ph ^= 1u;
            const int rows_here = min(R, m_rows - pass0);
            if (++s == S) s = 0;
            if (s == 0) w_ph ^= 1u;
            const unsigned char* xbuf = xs + (size_t)xb * R * x_stride;
            float* adjb = adjg + (size_t)xb * KB * R;
            if (fresh) {                               // new rows: each group forms its own copy of the corrections
                if (!mbar_wait(&x_full[xb], x_ph, abort_flag, p.status)) ok = false;
                // adj[kb][n] = -136 * sum of the row's activations over block kb (removes the code bias after the MMA);
                // a block is 16 chunks of 8 values: the 16 lanes of a half-warp hold one block of one row
                const int chunks_per_row = K >> 3;
                for (int nn = 0; nn < rows_here; ++nn) {
                    const unsigned char* xrow = xbuf + (size_t)nn * x_stride;
                    for (int base = cw * 32; base < chunks_per_row; base += kGroupThreads) {
                        const int ck = base + lane;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (ck < chunks_per_row) v = *reinterpret_cast<const uint4*>(xrow + ck * 16);
                        float sx = sum8_bf16(v);
#pragma unroll
                        for (int m = 8; m >= 1; m >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, m);
                        if (ck < chunks_per_row && (ck & 15) == 0) adjb[(ck >> 4) * R + nn] = -136.f * sx;
                    }
                }
                // rows beyond the group's last are zeroed once per staging (both consumer groups write the same zeros:
                // each reads them only after its own barrier below; no copy targets these rows until every warp
                // has released the buffer), so the fragment loads of the MMA loop need no row predicate
                for (int nn = rows_here; nn < R; ++nn) {
                    unsigned char* xrow = const_cast<unsigned char*>(xbuf) + (size_t)nn * x_stride;
                    for (int ck = cw * 32 + lane; ck < chunks_per_row; ck += kGroupThreads)
                        *reinterpret_cast<uint4*>(xrow + ck * 16) = make_uint4(0, 0, 0, 0);
                }
                group_sync(grp);
            }
            SPROF(long long c1 = clock64(); t_x += c1 - c0;)
            if (!mbar_wait(&w_full[s], w_ph, abort_flag, p.status)) ok = false;
            SPROF(long long c2 = clock64(); t_w += c2 - c1;)
            if ((n & 1) != grp) {                      // the other group's unit: nothing of this warp reads it
                if (lane == 0) {
                    mbar_arrive(&w_empty[s]);
                    if (x_done) mbar_arrive(&x_empty[xb]);             // this warp's earlier reads of the rows are complete
                }
                continue;
            }
            const unsigned char* stage = wst + (size_t)s * stage_bytes;
            float tot[NMW][NCH][4];
#pragma unroll
            for (int m = 0; m < NMW; ++m)
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                    for (int i = 0; i < 4; ++i) tot[m][ch][i] = 0.f;
#pragma unroll
            for (int b = 0; b < (FIXED ? BPWc : bpw); ++b) {
                const int kb = ks * bpw + b;
                uint4 wv[NMW][2];
                uint32_t sv[NMW];
#pragma unroll
                for (int m = 0; m < NMW; ++m) {
                    const int panel_local = GATEUP ? 2 * pp + (NMW == 2 ? m : mw) : pp;
                    const unsigned char* blk = stage + ((size_t)panel_local * KB + kb) * kBlockBytes;
                    wv[m][0] = *reinterpret_cast<const uint4*>(blk + lane * 16);
                    wv[m][1] = *reinterpret_cast<const uint4*>(blk + 512 + lane * 16);
                    sv[m] = *reinterpret_cast<const uint32_t*>(blk + kCodeBytes + q * 4);
                }
                // CHN independent accumulator chains per (matrix, chunk): the block's 8 MMAs would otherwise be one
                // dependent chain; the chains are added in fixed order below
                float acc[NMW][NCH][CHN][4];
#pragma unroll
                for (int m = 0; m < NMW; ++m)
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                        for (int cc = 0; cc < CHN; ++cc)
#pragma unroll
                            for (int i = 0; i < 4; ++i) acc[m][ch][cc][i] = 0.f;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int set = 0; set < 2; ++set) {
                        const int cc = (2 * h + set) % CHN;
                        const int k0 = kb * kGroup + 64 * h + 32 * set + 8 * c;
                        uint4 xv[NCH];
#pragma unroll
                        for (int ch = 0; ch < NCH; ++ch) {
                            xv[ch] = *reinterpret_cast<const uint4*>(xbuf + (size_t)(8 * ch + q) * x_stride + k0 * 2);
                        }
#pragma unroll
                        for (int m = 0; m < NMW; ++m) {
                            const uint32_t wq = set ? wv[m][h].z : wv[m][h].x;        // row q
                            const uint32_t wq8 = set ? wv[m][h].w : wv[m][h].y;       // row q + 8
                            uint32_t a0 = code_pair(wq, 0), a1 = code_pair(wq8, 0), a2 = code_pair(wq, 4), a3 = code_pair(wq8, 4);
#pragma unroll
                            for (int ch = 0; ch < NCH; ++ch) mma_m16n8k16(acc[m][ch][cc], a0, a1, a2, a3, xv[ch].x, xv[ch].y);
                            a0 = code_pair(wq, 8), a1 = code_pair(wq8, 8), a2 = code_pair(wq, 12), a3 = code_pair(wq8, 12);
#pragma unroll
                            for (int ch = 0; ch < NCH; ++ch) mma_m16n8k16(acc[m][ch][cc], a0, a1, a2, a3, xv[ch].z, xv[ch].w);
                        }
                    }
                float2 cr[NCH];
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
                    cr[ch] = *reinterpret_cast<const float2*>(adjb + (size_t)kb * R + 8 * ch + 2 * c);
#pragma unroll
                for (int m = 0; m < NMW; ++m) {        // post-scale the block's integer-valued sums (Eq. 3 scale)
                    const __half2 sc = *reinterpret_cast<const __half2*>(&sv[m]);
                    const float s_lo = __low2float(sc), s_hi = __high2float(sc);
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch) {
                        float sum[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            sum[i] = acc[m][ch][0][i];
#pragma unroll
                            for (int cc = 1; cc < CHN; ++cc) sum[i] += acc[m][ch][cc][i];
                        }
                        tot[m][ch][0] = fmaf(s_lo, sum[0] + cr[ch].x, tot[m][ch][0]);
                        tot[m][ch][1] = fmaf(s_lo, sum[1] + cr[ch].y, tot[m][ch][1]);
                        tot[m][ch][2] = fmaf(s_hi, sum[2] + cr[ch].x, tot[m][ch][2]);
                        tot[m][ch][3] = fmaf(s_hi, sum[3] + cr[ch].y, tot[m][ch][3]);
                    }
                }
            }
            // this warp is done with the weight stage, and with the rows when the next unit stages others
            __syncwarp();
            SPROF(long long c3 = clock64(); t_mma += c3 - c2; ++n_mine;)
            if (lane == 0) {
                mbar_arrive(&w_empty[s]);
                if (x_done) mbar_arrive(&x_empty[xb]);
            }
            if (!exchange) {
                // no K split and both matrices here: the warp finishes its panel from registers
                if (ok) {
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int nn = pass0 + 8 * ch + 2 * c + (i & 1);
                            if (nn >= m_rows) continue;
                            const int orow = (tile * PP + pp) * kPanelRows + q + 8 * (i >> 1);
                            if (GATEUP) {
                                const float gv = tot[0][ch][i], uv = tot[NMW - 1][ch][i];
                                p.act_out[(size_t)(row0 + nn) * a.I + orow] = __float2bfloat16_rn(gv / (1.f + __expf(-gv)) * uv);
                            } else {
                                const int pair = a.perm[row0 + nn];
                                p.y_out[(size_t)pair * a.H + orow] = p.topk_w[pair] * tot[0][ch][i];
                            }
                        }
                }
                continue;
            }
            // Partials cross shared memory once (buffer alternates with the group's units, so one barrier per unit
            // is enough); then warp j finishes the slices (panel, chunk, fragment word) = j, j + 8, ...: the sum
            // over the K ranges in ascending order, SwiGLU or routing weight, store.
            float* pb = part + (size_t)(grp * 2 + (mine_cnt & 1)) * part_words;
            ++mine_cnt;
#pragma unroll
            for (int m = 0; m < NMW; ++m) {
                const int mg = (NMW == 2) ? m : mw;                    // matrix index inside the tile
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        pb[((((pp * NM + mg) * KS + ks) * NCH + ch) * 4 + i) * 32 + lane] = tot[m][ch][i];
            }
            group_sync(grp);
            const int slices = PP * NCH * 4;
            for (int sl = cw; sl < slices; sl += kGroupWarps) {
                const int i = sl & 3, ch = (sl >> 2) % NCH, spp = sl / (4 * NCH);
                float v[NM];
#pragma unroll
                for (int mg = 0; mg < NM; ++mg) {
                    float acc1 = 0.f;
                    for (int s2 = 0; s2 < KS; ++s2)
                        acc1 += pb[((((spp * NM + mg) * KS + s2) * NCH + ch) * 4 + i) * 32 + lane];
                    v[mg] = acc1;
                }
                const int nn = pass0 + 8 * ch + 2 * c + (i & 1);
                if (nn >= m_rows || !ok) continue;
                const int orow = (tile * PP + spp) * kPanelRows + q + 8 * (i >> 1);
                if (GATEUP) {
                    const float gv = v[0], uv = v[NM - 1];
                    p.act_out[(size_t)(row0 + nn) * a.I + orow] = __float2bfloat16_rn(gv / (1.f + __expf(-gv)) * uv);
                } else {
                    const int pair = a.perm[row0 + nn];
                    p.y_out[(size_t)pair * a.H + orow] = p.topk_w[pair] * v[0];
                }
            }
            SPROF(t_ep += clock64() - c3;)
        }
        SPROF(if (blockIdx.x == 7 && lane == 0 && (cw == 0 || cw == 5))
                  printf("%s grp %d warp %d: units %d mine %d total %lld xwait %lld wwait %lld mma %lld epi %lld\n", GATEUP ? "gu" : "dn",
                         grp, cw, u1 - u0, n_mine, clock64() - t_begin, t_x, t_w, t_mma, t_ep);)
    }
}

template <int NCH, bool GATEUP>
bool launch_stream_cfg(const GemmArgs& a, const __nv_bfloat16* x, __nv_bfloat16* act, const float* w, float* y, int* status,
                       int max_groups, bool dependent, cudaStream_t st) {
    constexpr int NM = GATEUP ? 2 : 1;
    StreamGeom g;
    if (!stream_geometry(GATEUP ? a.H : a.I, GATEUP ? a.I : a.H, NM, NCH, &g)) return false;
    void (*kern)(const StreamArgs) = stream_gemm_kernel<NCH, GATEUP, 1>;
    int variant = 0;
    if (GATEUP && g.NMW == 2) {
        kern = stream_gemm_kernel<NCH, GATEUP, GATEUP ? 2 : 1>;
        variant = 1;
    }
#ifndef EXMOE_STREAM_GENERIC_ONLY
    // OLMoE's two matrices with their geometry as literals (d_model 2048: 16 blocks, one panel pair per tile, K in four
    // ranges; d_ff 1024: 8 blocks, four panels per tile, K in two ranges)
    const int KBv = (GATEUP ? a.H : a.I) / kGroup;
    if (GATEUP && g.NMW == 1 && KBv == 16 && g.PP == 1 && g.KS == 4) {
        kern = stream_gemm_kernel<NCH, GATEUP, 1, 16, 1, 4>;
        variant = 2;
    } else if (!GATEUP && KBv == 8 && g.PP == 4 && g.KS == 2) {
        kern = stream_gemm_kernel<NCH, GATEUP, 1, 8, 4, 2>;
        variant = 2;
    }
#endif
    static SmemOnce smem_once[3];
    allow_smem(kern, (int)kSmemLimit, smem_once[variant]);
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    StreamArgs p{};
    p.a = a;
    p.x_src = x;
    p.act_out = act;
    p.topk_w = w;
    p.y_out = y;
    p.status = status;
    p.PP = g.PP;
    p.KS = g.KS;
    p.n_stages = g.n_stages;
    p.n_xbuf = g.n_xbuf;
    p.stage_bytes = g.stage_bytes;
    p.x_stride = g.x_stride;
    p.off_x = (uint32_t)g.off_x;
    p.off_part = (uint32_t)g.off_part;
    p.off_adj = (uint32_t)g.off_adj;
    p.off_bar = (uint32_t)g.off_bar;
    const long long units = (long long)max_groups * g.tiles;          // the wave's units when every group takes one pass
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)(units < sms ? (units < 1 ? 1 : units) : sms));
    lc.blockDim = dim3(kStreamThreads);
    lc.dynamicSmemBytes = g.total;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = dependent ? 1 : 0;
    cudaLaunchKernelEx(&lc, kern, p);
    count_launch();
    return true;
}

}  // namespace

bool stream_supported(int H, int I) {
    StreamGeom g;
    return stream_geometry(H, I, 2, 1, &g) && stream_geometry(I, H, 1, 1, &g);
}

// One wave on the streaming kernels: eight rows of a group per pass.  (Sixteen rows per pass, NCH = 2, halve the
// shared-memory reads of the weights per row but double the MMAs of every unit; with a few rows per expert that
// measured slower at every batch size in this path's range.)
bool launch_stream_wave(const GemmArgs& a, const __nv_bfloat16* hidden, __nv_bfloat16* act, const float* topk_w, float* y,
                        int* status, int max_groups, bool gateup, bool down, cudaStream_t st) {
    bool ok = true;
#ifndef EXMOE_STREAM_NO_ENTRY_PDL
    const bool entry_dependent = true;
#else
    const bool entry_dependent = false;
#endif
#ifndef EXMOE_STREAM_NCH
#define EXMOE_STREAM_NCH 1
#endif
    if (gateup) ok = launch_stream_cfg<EXMOE_STREAM_NCH, true>(a, hidden, act, topk_w, y, status, max_groups, entry_dependent, st);
    // a programmatic dependent only when the gate/up kernel of the same wave was launched just before it
    if (down && ok) ok = launch_stream_cfg<EXMOE_STREAM_NCH, false>(a, act, act, topk_w, y, status, max_groups, gateup, st);
    return ok;
}

}  // namespace exmoe
