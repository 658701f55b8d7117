// Shared declarations of the exmoe CUDA library (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/exmoe.h"

namespace exmoe {

// ---- packed layout (Eq. 3 / Eq. 4): 16-row panels x 128-wide blocks of 1056 bytes -------------
constexpr int kGroup = 128;          // scale group along K
constexpr int kPanelRows = 16;       // rows per panel (one m16 MMA tile)
constexpr int kBlockBytes = 1056;    // 1024 code bytes + 16 FP16 scales
constexpr int kCodeBytes = 1024;

// bytes of a packed [rows, K] matrix
__host__ __device__ inline size_t matrix_bytes(int rows, int K) {
    return (size_t)(rows / kPanelRows) * (K / kGroup) * kBlockBytes;
}

// ---- plan buffers shared by the resolution, grouping and GEMM kernels ------------------------
// header words
enum { HDR_N_ACTIVE = 0, HDR_N_WAVES = 1, HDR_N_MISSES = 2, HDR_BAD_ID = 3, HDR_N_GROUPS = 4, HDR_N_VALID = 5,
       HDR_WORDS = 8 };

struct PlanPtrs {
    int32_t* header;        // [HDR_WORDS]
    int32_t* wave_of;       // [E]
    int32_t* slot_of;       // [E]
    int32_t* misses;        // [3*E] (expert, slot, wave)
    int32_t* key_miss;      // [n_keys] 1 where the group (wave, slot) holds an expert that missed in this call
    int n_keys;
    int32_t* counts;        // [n_keys]
    int32_t* offsets;       // [n_keys + 1]
    int32_t* group_keys;    // [n_keys] active keys, ascending
    int32_t* wave_start;    // [max_waves + 1] index into group_keys
    int32_t* perm;          // [max_pairs]
    int32_t* chunk_table;   // [n_keys][chunks] scratch of the chunked grouping (may be null)
    size_t chunk_table_words;
    int32_t* chunk_done;    // arrival counter of the chunked grouping (zero between calls)
};

struct LayerState {         // Section 3.3 state of one layer, device memory
    int32_t* expert_slot;   // [E]
    int32_t* slot_expert;   // [C]
    uint64_t* slot_stamp;   // [C]
    uint64_t* tick;         // [1]
    uint64_t* stats;        // [6] lookups, hits, misses, waves, h2d_bytes, forwards
};

struct GemmArgs {
    const uint8_t* slots;       // slot memory of the layer
    size_t slot_stride;         // bytes per slot
    const int32_t* counts;
    const int32_t* offsets;
    const int32_t* group_keys;
    const int32_t* wave_start;  // already offset to the wave: [0] first group, [1] end
    const int32_t* perm;
    const int32_t* key_miss;    // [n_keys] (see PlanPtrs); may be null
    int group_filter;           // 0 all groups of the wave; 1 only groups whose expert was resident; 2 only the missed ones
    int direct_keys;            // > 0: every key 0 .. direct_keys-1 is a (possibly empty) group of the call's only wave
                                // (all experts resident, key = expert id): kernels may read counts / offsets by key at
                                // once instead of going through wave_start and group_keys first
    int num_slots;              // C (key % C = slot)
    int top_k;
    int H, I;
};

// One wave of the small-problem path (decode): the GEMM kernels rebuild the grouping themselves.
struct SmallWave {
    const int32_t* ids;         // [n_pairs] top-k ids
    const int32_t* wave_of;     // null when C = E (slot = expert id, single wave)
    const int32_t* slot_of;
    int n_pairs, E, wave;
    PlanPtrs plan;              // published for the test hooks
    int* status;
    int* arrive;                // [T * H/16] zero-initialised arrival counters of the fused combine
    const __nv_bfloat16* hidden;
    __nv_bfloat16* act;
    const float* topk_w;
    float* y;
    __nv_bfloat16* out;
    int max_rows, max_groups;
    bool pairwise;              // T*k <= kPairMaxPairs and a single wave: per-pair gate/up, by-token down
    int32_t* saved_ids;         // [kPairMaxPairs]
};
constexpr int kPairMaxPairs = 32;
#ifndef EXMOE_SMALL_MAX_PAIRS
#define EXMOE_SMALL_MAX_PAIRS 24
#endif
constexpr int kSmallMaxPairs = EXMOE_SMALL_MAX_PAIRS;
constexpr int kSmallMaxSlots = 1024;

// launch accounting (exmoe_launch_count)
void count_launch(int n = 1);

// Raise a kernel's dynamic shared-memory limit once per device (function attributes are per device; the cache of
// "already done" is the caller's static SmemOnce, one per kernel instantiation).
struct SmemOnce { unsigned long long mask = 0; };
template <typename F>
inline bool allow_smem(F kern, int bytes, SmemOnce& once) {
    int dev = 0;
    const bool known = cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64;
    if (known && ((once.mask >> dev) & 1ull)) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (known) once.mask |= 1ull << dev;
    return true;
}

// ---- kernel launchers (defined in the .cu files) ------------------------------------------------
int* pack_flag_word();      // a device word for one exmoe_pack call's non-finite flag (no allocation)
int launch_pack(const exmoe_shape& s, const void* wg, const void* wu, const void* wd, void* out,
                int* d_flag, cudaStream_t st);
void launch_resolve(const exmoe_shape& s, int C, int Cw, size_t bytes_per_expert, const int32_t* ids, int n_pairs,
                    LayerState state, PlanPtrs plan, int* d_status, cudaStream_t st);
// Device-initiated miss path: one kernel copies wave `wave`'s missed experts from the mapped host bank into their slots.
void launch_fetch_misses(const PlanPtrs& plan, int wave, const uint8_t* bank_dev, uint8_t* slots, size_t bpe, int E, int C,
                         cudaStream_t st, bool small_grid = false, bool follows_resolve = true);
void launch_group(const exmoe_shape& s, int C, int n_keys, int max_waves, bool identity, const int32_t* ids,
                  int n_pairs, PlanPtrs plan, int* d_status, cudaStream_t st);
// Streaming kernels (bulk-copy weight ring in shared memory) for kSmallMaxPairs < T*k <= kStreamMaxPairs.
#ifndef EXMOE_STREAM_MAX_PAIRS
#define EXMOE_STREAM_MAX_PAIRS 640
#endif
constexpr int kStreamMaxPairs = EXMOE_STREAM_MAX_PAIRS;   // above: tensor-core path
bool stream_supported(int H, int I);
bool launch_stream_wave(const GemmArgs& a, const __nv_bfloat16* hidden, __nv_bfloat16* act, const float* topk_w, float* y,
                        int* status, int max_groups, bool gateup, bool down, cudaStream_t st);
void launch_small_wave(const GemmArgs& a, const SmallWave& w, cudaStream_t st, bool gateup, bool down);
bool pair_path_fits(int H, int I, int top_k);                           // shared memory of the per-pair kernels within limits
bool small_path_fits(int H, int I, int num_slots, int n_pairs);         // ... of the in-CTA-grouping kernels
size_t prefill_scratch_bytes(int max_pairs, int num_experts);
// CUtensorMap objects of the grouped hidden rows and of the activations, in device memory: per matrix a family of 16
// maps whose boxes hold 16, 32, ..., 256 rows (a tile's box holds exactly the rows its MMAs read); x family, then act
constexpr size_t kPrefillMapBytes = 2 * 16 * 128;
struct PrefillMaps { unsigned char* dev; };
int prefill_setup(PrefillMaps* maps, const __nv_bfloat16* xg, const __nv_bfloat16* act, int max_pairs, int H, int I);
void launch_wait_selftest(int* status, long long budget_cycles, int* result, cudaStream_t st);
// grouped copy of the hidden rows; when `single_wave` is given its CTA 0 also builds that wave's tile list in `scratch`
void launch_gather_rows(const __nv_bfloat16* hidden, const int32_t* perm, const int32_t* n_valid, int n_pairs, int top_k,
                        int H, __nv_bfloat16* xg, const GemmArgs* single_wave, const int32_t* wave_start, void* scratch,
                        bool small_n, cudaStream_t st);
// which: bit 0 = gate/up GEMM + SwiGLU, bit 1 = down GEMM x routing weight, bit 2 = (re)build the wave's tile list
// small_n: the 64-row, eight-stage kernel shape (a few dozen rows per expert) instead of the 256-row, four-stage one
void launch_prefill_wave(const GemmArgs& g, const int32_t* wave_start, void* scratch, int* status, const PrefillMaps* maps,
                         __nv_bfloat16* act, const float* topk_w, float* y, int which, bool small_n, cudaStream_t st);
#ifndef EXMOE_PREFILL_SMALL_N_MAX_PAIRS
#define EXMOE_PREFILL_SMALL_N_MAX_PAIRS 1024
#endif
constexpr int kPrefillSmallNMaxPairs = EXMOE_PREFILL_SMALL_N_MAX_PAIRS;
void launch_combine(const float* y, const int32_t* ids, int E, int T, int k, int H, __nv_bfloat16* out,
                    cudaStream_t st);

}  // namespace exmoe
