// Device-side expert-ID resolution with LRU slot replacement (Section 3.3), wave assignment and
// expert map with sentinel (Section 3.4 steps 1-2), and token grouping by (wave, slot): histogram,
// exclusive prefix sum and stable permutation of token-expert pairs (the grouping step of Figure 1's caption).
// Integer work only; every result is deterministic and bit-exact.
#include "common.cuh"

namespace exmoe {

// ------------------------------------------------------------------------------------------------
// Resolution: one CTA; warp 0 runs the (inherently sequential) LRU, with the argmin over slots
// spread over its lanes.
//   active list  = distinct valid ids, ascending
//   order        = resident-at-entry (ascending), then absent (ascending)
//   wave w       = order[w*Cw, (w+1)*Cw)
//   per wave: tick += 1; protect slots of members; hit -> stamp; miss -> evict the unprotected slot
//   with the smallest (stamp, index), install, stamp, protect.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
resolve_kernel(const int32_t* __restrict__ ids, int n_pairs, int E, int C, int Cw, unsigned long long bytes_per_expert,
               LayerState st, PlanPtrs plan, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned long long* s_stamp = reinterpret_cast<unsigned long long*>(smem_raw);       // [C]
    int* s_flag = reinterpret_cast<int*>(s_stamp + C);                                    // [E]
    int* s_order = s_flag + E;                                                            // [E]
    int* s_eslot = s_order + E;                                                           // [E]
    int* s_sexp = s_eslot + E;                                                            // [C]
    int* s_prot = s_sexp + C;                                                             // [C]
    __shared__ int s_bad;

    const int tid = threadIdx.x;
    // the miss-fetch kernel of the first wave may be placed now; it reads the plan only after this grid has completed
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) s_bad = 0;
    for (int e = tid; e < E; e += blockDim.x) {
        s_flag[e] = 0;
        s_eslot[e] = st.expert_slot[e];
        plan.wave_of[e] = -1;
        plan.slot_of[e] = -1;
    }
    for (int v = tid; v < C; v += blockDim.x) {
        s_sexp[v] = st.slot_expert[v];
        s_stamp[v] = st.slot_stamp[v];
    }
    if (plan.key_miss)
        for (int i = tid; i < plan.n_keys; i += blockDim.x) plan.key_miss[i] = 0;
    __syncthreads();
    for (int p = tid; p < n_pairs; p += blockDim.x) {
        const int id = ids[p];
        if (id >= 0 && id < E) s_flag[id] = 1;
        else s_bad = 1;
    }
    __syncthreads();
    if (tid >= 32) return;

    const int lane = tid;
    const unsigned lt = (1u << lane) - 1u;
    int n = 0;
    for (int pass = 0; pass < 2; ++pass) {                 // residents first, then absentees
        for (int base = 0; base < E; base += 32) {
            const int e = base + lane;
            const bool pred = e < E && s_flag[e] && ((s_eslot[e] >= 0) == (pass == 0));
            const unsigned b = __ballot_sync(0xffffffffu, pred);
            if (pred) s_order[n + __popc(b & lt)] = e;
            n += __popc(b);
        }
    }
    __syncwarp();
    const int n_waves = (n + Cw - 1) / Cw;
    unsigned long long tick = *st.tick;
    unsigned long long hits = 0, misses = 0;
    int nm = 0;
    for (int w = 0; w < n_waves; ++w) {
        ++tick;
        const int lo = w * Cw, hi = min(n, lo + Cw);
        for (int v = lane; v < C; v += 32) s_prot[v] = 0;
        __syncwarp();
        for (int i = lo + lane; i < hi; i += 32) {
            const int s = s_eslot[s_order[i]];
            if (s >= 0) s_prot[s] = 1;
        }
        __syncwarp();
        for (int i = lo; i < hi; ++i) {
            const int e = s_order[i];
            int s = s_eslot[e];
            if (s < 0) {
                unsigned long long best = ~0ull;
                int best_v = 0x7fffffff;
                for (int v = lane; v < C; v += 32) {
                    if (!s_prot[v] && (s_stamp[v] < best)) { best = s_stamp[v]; best_v = v; }   // ascending v: first min kept
                }
#pragma unroll
                for (int m = 16; m >= 1; m >>= 1) {
                    const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, m);
                    const int ov = __shfl_xor_sync(0xffffffffu, best_v, m);
                    if (ob < best || (ob == best && ov < best_v)) { best = ob; best_v = ov; }
                }
                s = best_v;
                if (lane == 0) {
                    const int old = s_sexp[s];
                    if (old >= 0) s_eslot[old] = -1;
                    s_sexp[s] = e;
                    s_eslot[e] = s;
                    s_prot[s] = 1;
                    plan.misses[3 * nm + 0] = e;
                    plan.misses[3 * nm + 1] = s;
                    plan.misses[3 * nm + 2] = w;
                    if (plan.key_miss) plan.key_miss[w * C + s] = 1;      // this group's weights arrive with the wave's fetch
                }
                ++nm;
                ++misses;
            } else {
                ++hits;
            }
            if (lane == 0) {
                s_stamp[s] = tick;
                plan.wave_of[e] = w;
                plan.slot_of[e] = s;
            }
            __syncwarp();
        }
    }
    for (int e = lane; e < E; e += 32) st.expert_slot[e] = s_eslot[e];
    for (int v = lane; v < C; v += 32) {
        st.slot_expert[v] = s_sexp[v];
        st.slot_stamp[v] = s_stamp[v];
    }
    if (lane == 0) {
        *st.tick = tick;
        st.stats[0] += (unsigned long long)n;
        st.stats[1] += hits;
        st.stats[2] += misses;
        st.stats[3] += (unsigned long long)n_waves;
        st.stats[4] += misses * bytes_per_expert;
        st.stats[5] += 1ull;
        plan.header[HDR_N_ACTIVE] = n;
        plan.header[HDR_N_WAVES] = n_waves;
        plan.header[HDR_N_MISSES] = nm;
        plan.header[HDR_BAD_ID] = s_bad;
        if (s_bad) atomicExch(status, EXMOE_ERR_BAD_EXPERT_ID);
    }
}

void launch_resolve(const exmoe_shape& s, int C, int Cw, size_t bytes_per_expert, const int32_t* ids, int n_pairs,
                    LayerState state, PlanPtrs plan, int* d_status, cudaStream_t st) {
    const int E = s.num_experts;
    const size_t smem = (size_t)C * 8 + (size_t)(3 * E + 2 * C) * 4;
    resolve_kernel<<<1, 256, smem, st>>>(ids, n_pairs, E, C, Cw, (unsigned long long)bytes_per_expert, state, plan,
                                        d_status);
    count_launch();
}

// ------------------------------------------------------------------------------------------------
// Device-initiated miss path (Section 3.4 step 3 without the host in the loop): the misses of one wave
// are fetched by this kernel straight from the pinned host bank, which the GPU reads over PCIe through
// its mapped address.  The miss list stays on the device, so the host neither waits for the plan nor
// issues a copy per expert, and the whole layer call is a fixed launch sequence (capturable in a CUDA
// graph even with C < E).  Stream order is the slot's ready flag: the kernel runs on the compute
// stream after every earlier reader of the slots it overwrites and before the wave's GEMM kernels.
//
// Work split: the wave's missed experts are cut into 32 KiB pieces handed round-robin to the CTAs;
// a thread has eight 16-byte loads in flight before its first store (256 threads x 8 x 16 B per CTA),
// which is what keeps the PCIe read pipeline full.
// ------------------------------------------------------------------------------------------------
constexpr int kFetchThreads = 256;
constexpr int kFetchVec = 8;
constexpr int kFetchPiece = kFetchThreads * kFetchVec * 16;           // 32,768 B

__global__ void __launch_bounds__(kFetchThreads)
fetch_misses_kernel(const int32_t* __restrict__ header, const int32_t* __restrict__ misses, int wave,
                    const uint8_t* __restrict__ bank, uint8_t* __restrict__ slots, unsigned long long bpe, int E, int C) {
    __shared__ int s_lo, s_hi;
    asm volatile("griddepcontrol.wait;" ::: "memory");  // launched as a programmatic dependent of the resolution kernel (wave 0)
    if (threadIdx.x == 0) {                            // the list is ordered by wave: this wave's entries are one run
        int n = header[HDR_N_MISSES];
        n = n < 0 ? 0 : (n > E ? E : n);
        int lo = 0;
        while (lo < n && misses[3 * lo + 2] < wave) ++lo;
        int hi = lo;
        while (hi < n && misses[3 * hi + 2] == wave) ++hi;
        s_lo = lo;
        s_hi = hi;
    }
    __syncthreads();
    const long long per = (long long)((bpe + kFetchPiece - 1) / kFetchPiece);
    const long long total = (long long)(s_hi - s_lo) * per;
    for (long long c = blockIdx.x; c < total; c += gridDim.x) {
        const int m = s_lo + (int)(c / per);
        const unsigned long long off = (unsigned long long)(c % per) * kFetchPiece;
        const int e = misses[3 * m], v = misses[3 * m + 1];
        if (e < 0 || e >= E || v < 0 || v >= C) continue;             // never leave the bank or the slot memory
        const unsigned long long left = bpe - off;
        const int n16 = (int)((left < (unsigned long long)kFetchPiece ? left : (unsigned long long)kFetchPiece) / 16);
        const int4* src = reinterpret_cast<const int4*>(bank + (size_t)e * bpe + off);
        int4* dst = reinterpret_cast<int4*>(slots + (size_t)v * bpe + off);
        int4 r[kFetchVec];
#pragma unroll
        for (int j = 0; j < kFetchVec; ++j) {
            const int i = threadIdx.x + kFetchThreads * j;
            if (i < n16) r[j] = __ldcs(src + i);
        }
#pragma unroll
        for (int j = 0; j < kFetchVec; ++j) {
            const int i = threadIdx.x + kFetchThreads * j;
            if (i < n16) __stcg(dst + i, r[j]);
        }
    }
}

void launch_fetch_misses(const PlanPtrs& plan, int wave, const uint8_t* bank_dev, uint8_t* slots, size_t bpe, int E, int C,
                         cudaStream_t st, bool small_grid, bool follows_resolve) {
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    cudaLaunchConfig_t lc{};
    // a prefetch runs beside another layer's GEMM kernels: 32 CTAs (1 MB of loads in flight) keep the host link
    // busy and leave the SMs to them
    lc.gridDim = dim3(small_grid ? 32 : 2 * sms);
    lc.blockDim = dim3(kFetchThreads);
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (wave == 0 && follows_resolve) ? 1 : 0;   // wave 0 directly follows the resolution kernel (same stream)
#ifdef EXMOE_DISABLE_PDL
    lc.numAttrs = 0;
#endif
    cudaLaunchKernelEx(&lc, fetch_misses_kernel, (const int32_t*)plan.header, (const int32_t*)plan.misses, wave, bank_dev, slots,
                       (unsigned long long)bpe, E, C);
    count_launch();
}

// ------------------------------------------------------------------------------------------------
// Grouping.  key(pair p) = wave_of[e]*C + slot_of[e]  (identity mode, C = E: key = e).
// Pairs with an invalid id are left out.  perm = pair indices ordered by key, ties by ascending p.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int pair_key(int id, int E, int C, bool identity, const int32_t* wave_of,
                                        const int32_t* slot_of) {
    if (id < 0 || id >= E) return -1;
    if (identity) return id;
    return wave_of[id] * C + slot_of[id];
}

// warp 0: exclusive scan of counts, list of active keys, first group of every wave, header
__device__ __forceinline__ void scan_keys_warp0(const int32_t* cnt, int n_keys, int C, int max_waves, PlanPtrs plan,
                                                int32_t* off_out, bool identity, int n_active_hint) {
    const int lane = threadIdx.x;
    const unsigned lt = (1u << lane) - 1u;
    int running = 0, ng = 0;
    for (int base = 0; base < n_keys; base += 32) {
        const int kx = base + lane;
        const int v = kx < n_keys ? cnt[kx] : 0;
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (kx < n_keys) {
            off_out[kx] = running + incl - v;
            plan.counts[kx] = v;
            plan.offsets[kx] = running + incl - v;
        }
        const unsigned b = __ballot_sync(0xffffffffu, v > 0);
        if (v > 0) plan.group_keys[ng + __popc(b & lt)] = kx;
        ng += __popc(b);
        running += __shfl_sync(0xffffffffu, incl, 31);
    }
    __syncwarp();
    __threadfence_block();
    if (lane == 0) {
        plan.offsets[n_keys] = running;
        off_out[n_keys] = running;
        plan.header[HDR_N_GROUPS] = ng;
        plan.header[HDR_N_VALID] = running;
        if (identity) {                                   // no resolution kernel ran: fill its header words
            plan.header[HDR_N_ACTIVE] = ng;
            plan.header[HDR_N_WAVES] = ng ? 1 : 0;
            plan.header[HDR_N_MISSES] = 0;
        }
    }
    __syncwarp();
    for (int w = lane; w <= max_waves; w += 32) {          // wave_start[w] = #active keys below w*C
        int c = 0;
        for (int g = 0; g < ng; ++g) c += (plan.group_keys[g] < w * C);
        plan.wave_start[w] = c;
    }
}

// Small problems (up to 2048 pairs): one CTA does histogram, scan and the stable permutation.
__global__ void __launch_bounds__(256)
group_small_kernel(const int32_t* __restrict__ ids, int n_pairs, int E, int C, int n_keys, int max_waves,
                   bool identity, PlanPtrs plan, int* __restrict__ status) {
    extern __shared__ __align__(16) int s_int[];
    int* s_cnt = s_int;                    // [n_keys]
    int* s_off = s_cnt + n_keys;           // [n_keys + 1]
    int* s_key = s_off + n_keys + 1;       // [n_pairs]
    __shared__ int s_bad;
    const int tid = threadIdx.x;
    // launched as a programmatic dependent of whatever precedes it in the stream (in a decode loop the previous layer
    // call's combine kernel): placed early, it waits here before it reads the ids
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // a kernel launched behind this one as a programmatic dependent may be placed now; it waits for this grid's
    // completion before it reads the plan
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) s_bad = 0;
    for (int i = tid; i < n_keys; i += blockDim.x) s_cnt[i] = 0;
    __syncthreads();
    for (int p = tid; p < n_pairs; p += blockDim.x) {
        const int key = pair_key(ids[p], E, C, identity, plan.wave_of, plan.slot_of);
        s_key[p] = key;
        if (key >= 0) atomicAdd(&s_cnt[key], 1);
        else s_bad = 1;
    }
    __syncthreads();
    if (tid < 32) scan_keys_warp0(s_cnt, n_keys, C, max_waves, plan, s_off, identity, 0);
    if (tid == 0 && s_bad) {
        plan.header[HDR_BAD_ID] = 1;
        atomicExch(status, EXMOE_ERR_BAD_EXPERT_ID);
    } else if (tid == 0 && identity) {
        plan.header[HDR_BAD_ID] = 0;
    }
    __syncthreads();
    // Stable placement, 256 pairs at a time in pair order: inside a warp equal keys are ranked by lane
    // (match_any), the warps of a chunk advance the per-key cursors (s_off, consumed here) one after the other.
    const int lane = tid & 31, warp = tid >> 5;
    for (int base = 0; base < n_pairs; base += 256) {
        const int p = base + tid;
        const int key = (p < n_pairs) ? s_key[p] : -1;
        const unsigned same = __match_any_sync(0xffffffffu, key);
        const int leader = __ffs(same) - 1;
        const int rank = __popc(same & ((1u << lane) - 1u));
        int pos0 = 0;
        for (int w = 0; w < 8; ++w) {
            if (warp == w && key >= 0 && lane == leader) {
                pos0 = s_off[key];
                s_off[key] = pos0 + __popc(same);
            }
            __syncthreads();
        }
        pos0 = __shfl_sync(0xffffffffu, pos0, leader);
        if (key >= 0) plan.perm[pos0 + rank] = p;
    }
}

// Large problems (prefill): histogram with global integer atomics ...
__global__ void __launch_bounds__(256)
group_hist_kernel(const int32_t* __restrict__ ids, int n_pairs, int E, int C, bool identity, PlanPtrs plan,
                  int* __restrict__ status) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n_pairs) return;
    const int key = pair_key(ids[p], E, C, identity, plan.wave_of, plan.slot_of);
    if (key >= 0) atomicAdd(&plan.counts[key], 1);
    else {
        plan.header[HDR_BAD_ID] = 1;
        atomicExch(status, EXMOE_ERR_BAD_EXPERT_ID);
    }
}

// ... then one CTA per key compacts its pairs in ascending pair order (stable by construction).
// CTA 0 also publishes offsets, the active-key list and the per-wave ranges.
__global__ void __launch_bounds__(256)
group_scatter_kernel(const int32_t* __restrict__ ids, int n_pairs, int E, int C, int n_keys, int max_waves,
                     bool identity, PlanPtrs plan, const int32_t* __restrict__ hist) {
    extern __shared__ __align__(16) int s_int[];           // CTA 0: [n_keys + 1] scratch offsets
    __shared__ int s_warp[8];
    __shared__ int s_base;
    const int key = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cnt = hist[key];
    if (key == 0 && tid < 32) scan_keys_warp0(hist, n_keys, C, max_waves, plan, s_int, identity, 0);
    if (cnt == 0) return;
    if (warp == 0) {                                       // my offset = sum of counts below my key
        int acc = 0;
        for (int i = lane; i < key; i += 32) acc += hist[i];
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
        if (lane == 0) s_base = acc;
    }
    __syncthreads();
    int running = s_base;
    for (int base = 0; base < n_pairs; base += 256 * 4) {
        const int p0 = base + tid * 4;
        int f[4], c = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int p = p0 + j;
            f[j] = (p < n_pairs) && (pair_key(ids[p], E, C, identity, plan.wave_of, plan.slot_of) == key);
            c += f[j];
        }
        int incl = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int wbase = 0, total = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const int v = s_warp[w];
            if (w < warp) wbase += v;
            total += v;
        }
        int pos = running + wbase + incl - c;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (f[j]) plan.perm[pos++] = p0 + j;
        running += total;
        __syncthreads();
    }
}


// Large problems, second scheme (used when the scratch fits): the pairs are cut into chunks of 512.
//   kernel 1: one CTA per chunk histograms its pairs in shared memory and publishes count[key][chunk]; the last CTA
//             to finish (arrival counter, no spin) turns the table into absolute bases: offsets[key] from the
//             scan over keys, then the exclusive scan over the chunks of each key.
//   kernel 2: one CTA per chunk places its pairs: rank inside the warp from match_any, warps take their turn in
//             order to advance a shared-memory cursor per key, so equal keys keep ascending pair order (stable).
constexpr int kChunk = 512;
#ifndef EXMOE_GROUP_SMALL_MAX
#define EXMOE_GROUP_SMALL_MAX 2048
#endif

__global__ void __launch_bounds__(kChunk)
group_chunk_count_kernel(const int32_t* __restrict__ ids, int n_pairs, int E, int C, int n_keys, int max_waves,
                         bool identity, PlanPtrs plan, int32_t* __restrict__ table, int32_t* __restrict__ done,
                         int* __restrict__ status) {
    extern __shared__ __align__(16) int s_hist[];          // [n_keys] (+ [n_keys + 1] scratch offsets for the last CTA)
    __shared__ int s_last, s_bad;
    const int tid = threadIdx.x, chunk = blockIdx.x, n_chunks = gridDim.x;
    if (tid == 0) s_bad = 0;
    for (int i = tid; i < n_keys; i += kChunk) s_hist[i] = 0;
    __syncthreads();
    const int p = chunk * kChunk + tid;
    if (p < n_pairs) {
        const int key = pair_key(ids[p], E, C, identity, plan.wave_of, plan.slot_of);
        if (key >= 0) atomicAdd(&s_hist[key], 1);
        else s_bad = 1;
    }
    __syncthreads();
    for (int i = tid; i < n_keys; i += kChunk) table[(size_t)i * n_chunks + chunk] = s_hist[i];
    if (tid == 0 && s_bad) {
        plan.header[HDR_BAD_ID] = 1;
        atomicExch(status, EXMOE_ERR_BAD_EXPERT_ID);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(done, 1) == n_chunks - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) *done = 0;                               // ready for the next call
    // totals per key -> plan.counts (one warp per key, lanes over chunks); warp 0 then scans the keys
    const int lane = tid & 31, warp = tid >> 5;
    for (int i = warp; i < n_keys; i += kChunk / 32) {
        int tot = 0;
        for (int c = lane; c < n_chunks; c += 32) tot += __ldcg(&table[(size_t)i * n_chunks + c]);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, m);
        if (lane == 0) {
            plan.counts[i] = tot;
            s_hist[i] = tot;
        }
    }
    __syncthreads();
    int* s_off = s_hist + n_keys;
    if (tid < 32) scan_keys_warp0(s_hist, n_keys, C, max_waves, plan, s_off, identity, 0);
    __syncthreads();
    for (int i = warp; i < n_keys; i += kChunk / 32) {     // absolute base of every (key, chunk): exclusive scan over chunks
        int running = s_off[i];
        for (int c0 = 0; c0 < n_chunks; c0 += 32) {
            const int c = c0 + lane;
            const int v = c < n_chunks ? __ldcg(&table[(size_t)i * n_chunks + c]) : 0;
            int incl = v;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += o;
            }
            if (c < n_chunks) table[(size_t)i * n_chunks + c] = running + incl - v;
            running += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
}

__global__ void __launch_bounds__(kChunk)
group_chunk_scatter_kernel(const int32_t* __restrict__ ids, int n_pairs, int E, int C, int n_keys, bool identity,
                           PlanPtrs plan, const int32_t* __restrict__ table) {
    extern __shared__ __align__(16) int s_cur[];           // [n_keys] pairs of this chunk already placed, per key
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, chunk = blockIdx.x, n_chunks = gridDim.x;
    for (int i = tid; i < n_keys; i += kChunk) s_cur[i] = 0;
    const int p = chunk * kChunk + tid;
    int key = -1;
    if (p < n_pairs) key = pair_key(ids[p], E, C, identity, plan.wave_of, plan.slot_of);
    const unsigned same = __match_any_sync(0xffffffffu, key);
    const int rank = __popc(same & ((1u << lane) - 1u));
    const bool leader = key >= 0 && rank == 0;
    __syncthreads();
    int base = 0;
    for (int w = 0; w < kChunk / 32; ++w) {                // warps in order: ascending pair index
        if (warp == w && leader) {
            base = s_cur[key];
            s_cur[key] = base + __popc(same);
        }
        __syncthreads();
    }
    base = __shfl_sync(0xffffffffu, base, __ffs(same) - 1);
    if (key >= 0) plan.perm[table[(size_t)key * n_chunks + chunk] + base + rank] = p;
}

void launch_group(const exmoe_shape& s, int C, int n_keys, int max_waves, bool identity, const int32_t* ids,
                  int n_pairs, PlanPtrs plan, int* d_status, cudaStream_t st) {
    const int E = s.num_experts;
    if (n_pairs <= EXMOE_GROUP_SMALL_MAX && n_keys <= 4096) {
        const size_t smem = (size_t)(2 * n_keys + 1 + n_pairs) * 4;
        static SmemOnce smem_once;
        allow_smem(group_small_kernel, 64 * 1024, smem_once);
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3(1);
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
        cudaLaunchKernelEx(&lc, group_small_kernel, ids, n_pairs, E, C, n_keys, max_waves, identity, plan, d_status);
        count_launch();
        return;
    }
    const int n_chunks = (n_pairs + kChunk - 1) / kChunk;
    if (plan.chunk_table && (size_t)n_keys * n_chunks <= plan.chunk_table_words && n_keys <= 5000) {
        if (identity) cudaMemsetAsync(plan.header + HDR_BAD_ID, 0, 4, st);
        group_chunk_count_kernel<<<n_chunks, kChunk, (size_t)(2 * n_keys + 1) * 4, st>>>(
            ids, n_pairs, E, C, n_keys, max_waves, identity, plan, plan.chunk_table, plan.chunk_done, d_status);
        group_chunk_scatter_kernel<<<n_chunks, kChunk, (size_t)n_keys * 4, st>>>(ids, n_pairs, E, C, n_keys, identity, plan,
                                                                               plan.chunk_table);
        count_launch(2);
        return;
    }
    // counts doubles as the histogram; it is rewritten with the same values by CTA 0's scan
    cudaMemsetAsync(plan.counts, 0, (size_t)n_keys * 4, st);
    if (identity) cudaMemsetAsync(plan.header + HDR_BAD_ID, 0, 4, st);
    group_hist_kernel<<<(n_pairs + 255) / 256, 256, 0, st>>>(ids, n_pairs, E, C, identity, plan, d_status);
    group_scatter_kernel<<<n_keys, 256, (size_t)(n_keys + 1) * 4, st>>>(ids, n_pairs, E, C, n_keys, max_waves,
                                                                      identity, plan, plan.counts);
    count_launch(2);
}

}  // namespace exmoe
