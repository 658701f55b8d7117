/*
 * exmoe.h - C ABI of the B200 (sm_100a) complete-expert sparse-MoE layer forward.
 *
 * What the library computes (ExactMoE paper, Section 3):
 *   Eq. 2    y_t = sum_{e in TopK_t} p_{t,e} * W_d,e [ silu(W_g,e h_t) (.) W_u,e h_t ]
 *   Eq. 3    routed expert weights are symmetric group-128 int4: s = absmax/7,
 *            q = clip(round(W/s), -8, 7), W^ = s*q defines the arithmetic; FP16 scales.
 *   Sec. 3.3 every layer owns C expert slots (k <= C <= E) holding the packed bytes; the same
 *            bytes live in a pinned host bank; a miss is one asynchronous copy; LRU replacement
 *            among slots the current wave does not use; C = E preloads and bypasses lookups.
 *   Sec. 3.4 the active expert set is cut into waves of at most `wave_cap` experts; per wave:
 *            resolve/load, expert map with sentinel, fused grouped gate/up GEMM + SwiGLU and down
 *            GEMM over the complete token matrix, accumulate, completion event.
 *
 * Conventions
 *   - Every entry point returns an int status: EXMOE_OK (0) or a negative EXMOE_ERR_* code.
 *     Nothing throws, aborts or traps the device.  exmoe_strerror() names a code.
 *   - "dev" pointers are device memory of the current CUDA device, "host" pointers are host
 *     memory.  `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - The caller owns every buffer it passes (tensors, slot memory, workspace, host bank) and
 *     must keep them alive while the cache exists.  The library owns only its host bookkeeping,
 *     one copy stream, its events, pinned staging buffers and the graphs of exmoe_moe_forward_host.
 *   - BF16 tensors are row-major, dense.  ids are int32, mixture weights are float32.
 *   - All calls on one cache must come from one host thread at a time, and all forwards (and prefetches of the same
 *     layer) on one cache must be issued to ONE stream or be ordered by the caller with events: the workspace
 *     (plan, activations, pair buffer) is shared by the layers, and the host-copy miss path orders slot reuse against
 *     the stream that ran the earlier wave.
 */
#ifndef EXMOE_H
#define EXMOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    EXMOE_OK = 0,
    EXMOE_ERR_ARG = -1,           /* null pointer, negative size, T > max_tokens, layer out of range */
    EXMOE_ERR_SHAPE = -2,         /* d_model or d_ff not a multiple of 128 (Sec. 7 leaves such shapes to padding), group_size
                                     != 128, top_k > num_slots, num_slots > num_experts (Sec. 3.3), a size beyond a kernel's
                                     shared memory */
    EXMOE_ERR_NOT_PINNED = -3,    /* a host bank pointer is not page-locked host memory (Sec. 3.3) */
    EXMOE_ERR_CUDA = -4,          /* a CUDA runtime call failed */
    EXMOE_ERR_NONFINITE = -5,     /* exmoe_pack: a weight is NaN/Inf or a scale overflows FP16 */
    EXMOE_ERR_BAD_EXPERT_ID = -6, /* a top-k id was outside [0, E); that pair contributed nothing */
    EXMOE_ERR_TIMEOUT = -7,       /* a bounded device-side wait expired */
    EXMOE_ERR_STATE = -8          /* call order: e.g. debug plan asked for a layer that did not run last */
};

/* Geometry of one sparse layer (Sec. 4.1 gives OLMoE's: 2048, 1024, 64, 8).  group_size must be 128. */
typedef struct {
    int d_model;      /* H: hidden size, K of gate/up, N of down */
    int d_ff;         /* I: expert intermediate size */
    int num_experts;  /* E */
    int top_k;        /* k */
    int group_size;   /* 128 (Eq. 3) */
} exmoe_shape;

/* Runtime counters of one layer's cache: the quantities the cache reports in Sec. 4.2 and Table 1 (hit rate, host-to-
 * device traffic).  All zero while the layer is fully resident (C = E): no lookups happen then (Sec. 3.3, Fig. 2 caption). */
typedef struct {
    uint64_t lookups;    /* active experts looked up, summed over calls */
    uint64_t hits;
    uint64_t misses;
    uint64_t waves;
    uint64_t h2d_bytes;  /* misses * bytes of one packed expert */
    uint64_t forwards;   /* layer calls */
} exmoe_stats;

typedef struct exmoe_cache exmoe_cache; /* opaque */

/* Name of a status code (no paper counterpart: part of this ABI's error convention).  Never NULL. */
const char* exmoe_strerror(int code);

/* Eq. 4: bytes of one packed expert = 3*I*H * (4/8 + 16/(128*8)); 3,244,032 for OLMoE.
 * This is also the size of one GPU slot and of one entry of the host bank. */
int exmoe_packed_bytes(const exmoe_shape* shape, size_t* bytes_per_expert);

/* Offline conversion of ONE expert (Eq. 3 + this library's packed layout, Sec. 3.2).
 *   w_gate_bf16, w_up_bf16 : dev, BF16 [I, H]     w_down_bf16 : dev, BF16 [H, I]
 *   packed_out             : dev, bytes_per_expert, 16-byte aligned
 * Layout: 16-row panels x 128-wide blocks of 1056 bytes (1024 bytes of offset-binary nibbles in
 * the register order of the kernels, then 16 FP16 scales); gate and up panels alternate, the down
 * matrix follows.  Quantiser: binary32 absmax, s = fp16(absmax/7), q = clip(rint(W/s), -8, 7) with
 * IEEE division and round-half-even; a zero (or FP16-underflowing) group has s = 0, q = 0.
 * Runs on `stream` and waits for it, so the status covers the data: EXMOE_ERR_NONFINITE if any
 * weight is NaN/Inf or a scale overflows FP16 (the output is then unspecified). */
int exmoe_pack(const exmoe_shape* shape, const void* w_gate_bf16, const void* w_up_bf16,
               const void* w_down_bf16, void* packed_out, void* stream);

/* Sizes of the two device buffers the caller must allocate for exmoe_cache_create (Sec. 3.3):
 *   slot_bytes_total = num_layers * num_slots * bytes_per_expert
 *   workspace_bytes  = cache state + plan + token grouping + intermediate activations for
 *                      up to max_tokens tokens per call. */
int exmoe_cache_workspace_bytes(const exmoe_shape* shape, int num_layers, int num_slots,
                                int max_tokens, size_t* slot_bytes_total, size_t* workspace_bytes);

/* Create the slot caches of `num_layers` sparse layers, C = num_slots slots each (Sec. 3.3).
 *   host_bank[l] : host, pinned, E * bytes_per_expert bytes: expert e of layer l at offset
 *                  e * bytes_per_expert, exactly as exmoe_pack wrote it.
 *   slot_mem     : dev, slot_bytes_total, 256-byte aligned.   workspace : dev, workspace_bytes, 256-aligned.
 *   wave_cap     : experts per wave, 1..num_slots; 0 means num_slots (a wave never exceeds C, Sec. 3.4).
 * C = E: all experts are copied into their slots here (slot = expert id) and later calls do no
 * lookups.  C < E: the cache starts empty.  Synchronous. */
int exmoe_cache_create(exmoe_cache** out, const exmoe_shape* shape, int num_layers, int num_slots,
                       const void* const* host_bank, void* slot_mem, void* workspace,
                       int max_tokens, int wave_cap);

/* One sparse-layer forward (Eq. 2 through Sec. 3.4's waves).
 *   hidden_bf16  : dev, BF16 [T, H]        topk_ids : dev, int32 [T, k]
 *   topk_weights : dev, float32 [T, k]     out_bf16 : dev, BF16 [T, H], fully overwritten
 * Mixture weights are used as given (no renormalisation, Sec. 3.4).  Pair contributions are
 * accumulated in binary32 in the order j = 0..k-1 and rounded once to BF16, so the result does not
 * depend on C, wave_cap or cache history.  T = 0 is a no-op.  An id outside [0, E) contributes
 * nothing and sets the sticky status EXMOE_ERR_BAD_EXPERT_ID (see exmoe_status).
 * C = E: fully asynchronous on `stream`.  C < E: see exmoe_cache_set_miss_path; with the default
 * device-initiated miss path the call is fully asynchronous on `stream` as well.
 * With all experts resident and T * k <= 2048 the call's first kernel (gate/up of the smallest calls, grouping of the
 * others) is launched with programmatic stream serialisation: its blocks may be placed while the
 * kernel before it in `stream` still runs (if that kernel releases its dependents early, as this library's last
 * kernels do), but it reads and writes nothing before that kernel has completed: stream order holds for memory. */
int exmoe_moe_forward(exmoe_cache* cache, int layer, const void* hidden_bf16, const int32_t* topk_ids,
                      const float* topk_weights, int T, void* out_bf16, void* stream);

/* The same layer call for a caller whose tensors live in HOST memory (pageable or pinned):
 *   hidden_host : host, BF16 [T, H]      ids_host : host, int32 [T, k]      weights_host : host, float32 [T, k]
 *   out_host    : host, BF16 [T, H], fully overwritten
 * The inputs are copied into the library's pinned staging buffer, go to the device in one copy, the layer runs as
 * in exmoe_moe_forward, the result comes back in one copy (results of up to 64 KB are written by the last kernel
 * straight into the pinned staging buffer), and the call returns when out_host holds it (synchronous; `stream`
 * carries the work).  Tiny batches (T * top_k <= 24) whose call contains no host wait (C = E, or the
 * device-initiated miss path) record their launch sequence once per (layer, T) in a CUDA graph and replay it; all
 * other calls issue their launches one by one.  Calls of 256 KB of activations or more whose four tensors are
 * page-locked skip the staging buffer: the device copies use the caller's memory.  Same results, state and errors
 * as exmoe_moe_forward.  Not to be called while `stream` is being captured by the caller. */
int exmoe_moe_forward_host(exmoe_cache* cache, int layer, const void* hidden_host, const int32_t* ids_host,
                           const float* weights_host, int T, void* out_host, void* stream);

/* How the misses of a C < E cache reach their slots (Sec. 3.4 step 3; the paper's runtime issues host copies).
 *   EXMOE_MISS_DEVICE_FETCH (default when every host bank has a 16-byte aligned device-visible address, which
 *       page-locked memory of cudaHostAlloc / cudaHostRegister has): the miss list stays on the device; before each
 *       wave's GEMM kernels a kernel on the caller's stream reads the wave's missed experts straight out of the
 *       pinned host bank (through its mapped address, over PCIe) into their slots.  The host waits for nothing and
 *       exmoe_moe_forward is a fixed launch sequence that may be captured in a CUDA graph.  It launches
 *       ceil(min(T*k, E) / wave_cap) waves whatever the ids turn out to be (a wave without work finds none).  For
 *       24 < T*k <= 640 the fetch kernel runs on the library's side stream while the wave's GEMM kernels run over the
 *       groups whose experts were already resident; the kernels over the fetched groups wait for it (events in both
 *       directions, inside the capture too).  Smaller and larger calls fetch and compute in stream order.
 *   EXMOE_MISS_HOST_COPIES: the resolution kernel's miss plan is read back once per call (the paper's single
 *       batched id transfer) and the host waits for it, then issues one copy per missed expert on the library's
 *       copy stream, ordered against the compute stream by events; the copies of a wave overlap the kernels of
 *       the wave before it, and the call returns before they finish.  Not capturable.
 * Outputs, cache state and statistics are identical in both modes.  The call synchronises the device, so the
 * switch is ordered against earlier calls.  EXMOE_ERR_NOT_PINNED if device fetch is asked for and a bank has no
 * such address; the mode is then unchanged.  No effect when C = E. */
enum { EXMOE_MISS_HOST_COPIES = 0, EXMOE_MISS_DEVICE_FETCH = 1 };
int exmoe_cache_set_miss_path(exmoe_cache* cache, int mode);

/* Prefetch (the paper cites prefetching as related work and leaves it out; Sec. 3.3's slot map is what it acts on).
 * Treats `expert_ids` (dev, int32 [n_ids], any order, repeats allowed, n_ids <= max_tokens * top_k) as the ids of a
 * layer call without tokens: the slot map, LRU stamps, waves and counters of `layer` advance exactly as in
 * Sec. 3.3 / 3.4 steps 1-3 for those ids (hits are stamped, misses evict the least recently used unprotected slots
 * and are fetched from the host bank), and nothing is computed.  A later exmoe_moe_forward that selects these
 * experts then finds them resident.  Outputs never depend on the cache state, so a wrong guess costs transfer time
 * and slots, not correctness.  Asynchronous on `stream`; uses its own resolution buffers, so it may run beside an
 * exmoe_moe_forward of ANOTHER layer on another stream; calls on the same layer (prefetch or forward) must be
 * ordered by the caller (same stream, or events).  Needs the device-initiated miss path (EXMOE_ERR_STATE
 * otherwise); no-op when C = E or n_ids = 0.  An id outside [0, E) is ignored and sets the sticky status
 * EXMOE_ERR_BAD_EXPERT_ID. */
int exmoe_cache_prefetch(exmoe_cache* cache, int layer, const int32_t* expert_ids, int n_ids, void* stream);

/* Router of one sparse block (Eq. 1; the selected probabilities are used as they are, Sec. 3.4): logits z_t = W_r h_t in
 * binary32 (BF16 products, fixed summation order), plus `bias` if given, softmax over all E experts, the k
 * largest, equal values ordered by ascending expert id.  Writes exmoe_moe_forward's inputs on the device.
 *   hidden_bf16  : dev, BF16 [T, H], 16-byte aligned     router_bf16 : dev, BF16 [E, H], 16-byte aligned
 *   bias         : dev, float32 [E], or NULL
 *   topk_ids     : dev, int32 [T, k], descending probability     topk_weights : dev, float32 [T, k]
 * Uses shape->d_model (a multiple of 8), num_experts (<= 4096) and top_k; asynchronous on `stream`;
 * allocates nothing; T = 0 is a no-op.  EXMOE_ERR_SHAPE / EXMOE_ERR_ARG before any work is queued. */
int exmoe_route(const exmoe_shape* shape, const void* hidden_bf16, const void* router_bf16, const float* bias,
                int T, int32_t* topk_ids, float* topk_weights, void* stream);

/* Tiny-batch forward that allocates nothing and needs no cache object (the paper has no counterpart: this
 * is a service for one kind of caller, not a step of the method).
 *
 * Who it is for: code that cannot get device memory at the moment it needs this layer - a serving loop that
 * handed all device memory to its own pool at start-up, a plug-in living under a host framework that owns the
 * allocator, or a latency-critical path that must not pay the device-wide synchronisation a cudaMalloc or
 * cudaFree brings.  exmoe_moe_forward needs a caller-allocated workspace for the activations that travel from
 * the gate/up kernel to the down kernel; here that scratch is a fixed 262,400-byte `__device__` array inside
 * the library (held by every GPU that loads the library until the process exits), so the caller passes inputs
 * and outputs only.  The function calls no cudaMalloc, cudaFree or other allocating routine.
 *
 *   experts_dev  : dev, num_experts packed experts back to back (expert e at e * bytes_per_expert), i.e. a
 *                  fully resident layer exactly as exmoe_pack wrote it (slot = expert id, one wave).
 *   hidden_bf16, topk_ids, topk_weights, out_bf16 : as for exmoe_moe_forward.  These are the kernels
 *                  exmoe_moe_forward runs for T * top_k <= 24 on a fully resident layer, and there the two
 *                  entry points return the same bits; for 24 < T * top_k <= 32 exmoe_moe_forward switches to
 *                  its streaming kernels, which split K differently, and the two agree within the output
 *                  tolerance (a few BF16 roundings), not bit for bit.
 *
 * Limits: T * top_k <= 32 and d_ff <= 4096 (the size of the scratch), and the shared memory of the two kernels:
 * top_k * (2 * d_ff + 132 + d_ff / 32) <= 204,800 bytes and 2 * d_model + d_model / 32 + 7,232 <= 102,400 bytes
 * (d_ff = 4096 allows top_k <= 24; OLMoE's 1024 allows 32); anything larger is refused with EXMOE_ERR_SHAPE before
 * any work is queued.  T = 0 is a no-op.
 * First call on a device: looks up the device address of the scratch array (cudaGetSymbolAddress, with that
 * device current) and keeps it; make this first call outside any stream capture.
 * The scratch is shared by all calls and keeps the previous call's contents; the function clears the one word
 * that must start at zero.  Calls on one device that may overlap on the GPU (different streams without
 * ordering between them) race on it: order them, or use exmoe_moe_forward with separate workspaces.
 * An id outside [0, E) contributes nothing.  What the kernels find on the device - such an id
 * (EXMOE_ERR_BAD_EXPERT_ID) or a bounded wait that expired (EXMOE_ERR_TIMEOUT, output rows then unwritten) - cannot be
 * returned by this asynchronous call: it is kept in a sticky word of the scratch and read with
 * exmoe_moe_forward_static_status(). */
int exmoe_moe_forward_static(const exmoe_shape* shape, const void* experts_dev, const void* hidden_bf16,
                             const int32_t* topk_ids, const float* topk_weights, int T, void* out_bf16,
                             void* stream);

/* Sticky device-side status of exmoe_moe_forward_static on the current device (the paper has no counterpart):
 * synchronises the device, returns EXMOE_OK or the last EXMOE_ERR_BAD_EXPERT_ID / EXMOE_ERR_TIMEOUT recorded since the
 * previous call of this function, and clears it.  Allocates nothing. */
int exmoe_moe_forward_static_status(void);

/* Test hooks (synchronise).  Sec. 3.3 state of one layer: expert_slot [E] (-1 = not resident),
 * slot_expert [C] (-1 = empty), slot_stamp [C], all host pointers, any may be NULL. */
int exmoe_cache_get_state(exmoe_cache* cache, int layer, int32_t* expert_slot, int32_t* slot_expert,
                          uint64_t* slot_stamp, uint64_t* tick);

/* Plan of the most recent exmoe_moe_forward, which must have been for `layer` (Sec. 3.4 steps 1-2
 * and the token grouping): wave_of [E], slot_of [E] (-1 = inactive sentinel), counts [n_keys],
 * offsets [n_keys + 1], perm [T*k] (first offsets[n_keys] entries valid), misses [3*E] as
 * (expert, slot, wave) triples; n_keys = ceil(E / wave_cap) * C.  Any output pointer may be NULL. */
int exmoe_debug_last_plan(exmoe_cache* cache, int layer, int32_t* n_active, int32_t* n_waves,
                          int32_t* n_misses, int32_t* wave_of, int32_t* slot_of, int32_t* counts,
                          int32_t* offsets, int32_t* perm, int32_t* misses);

/* Which kernel family served the most recent exmoe_moe_forward of this cache (test and measurement hook; the paper
 * has no counterpart: Sec. 3.4 only says "two grouped GEMMs per wave").  The choice depends on T * top_k, on the
 * number of waves and on whether the shape fits the kernel, never on the values of the tensors.  Returns one of
 * EXMOE_PATH_* (positive), EXMOE_ERR_STATE before the first forward.  Does not synchronise. */
enum {
    EXMOE_PATH_PAIR = 2,           /* per-pair gate/up kernel + by-token down kernel (T*k <= 24, one wave) */
    EXMOE_PATH_SMALL = 3,          /* grouping rebuilt inside the GEMM CTAs (T*k <= 24, several waves) */
    EXMOE_PATH_STREAM = 4,         /* bulk-copy weight ring + register dequantisation (T*k <= 640) */
    EXMOE_PATH_TENSOR_SMALL_N = 5, /* tcgen05 kernels, 64-row token tiles (T*k <= 1024) */
    EXMOE_PATH_TENSOR = 6          /* tcgen05 kernels, 256-row token tiles */
};
int exmoe_debug_last_path(exmoe_cache* cache);

/* Bytes of the staged host-to-device input copy of the most recent exmoe_moe_forward_host (test hook; no paper
 * counterpart): T * d_model * 2 + 2 * T * top_k * 4 rounded up to 16-byte pieces, whatever max_tokens is. */
int exmoe_debug_last_host_copy_bytes(exmoe_cache* cache, size_t* h2d_bytes);

/* Copy one slot's bytes back to the host (test hook for the miss-copy path; synchronises). */
int exmoe_debug_read_slot(exmoe_cache* cache, int layer, int slot, void* host_out);

/* Failure-detection self-test (no paper counterpart).  Every device-side wait in this library is bounded: when
 * its budget of clock ticks runs out the waiting code raises the sticky status EXMOE_ERR_TIMEOUT, the CTA's
 * roles leave their loops, tensor memory is released and the kernel returns, so the context stays usable.
 * This hook runs a one-warp kernel that waits, with a budget of `budget_cycles` SM clock ticks (1..4e9), on a
 * barrier that nothing completes.  *gave_up gets bit 0 = the wait returned "expired", bit 1 = the abort flag was
 * raised; exmoe_status() then reports EXMOE_ERR_TIMEOUT.  Synchronous. */
int exmoe_debug_wait_timeout(exmoe_cache* cache, long long budget_cycles, int* gave_up);

/* Counters of one layer's cache (Sec. 4.2: hit rate and transferred bytes are reported per configuration).  Synchronises. */
int exmoe_cache_stats(exmoe_cache* cache, int layer, exmoe_stats* out);
/* Back to the state after exmoe_cache_create: empty cache (C < E), zero stamps and counters (Sec. 3.3 start state;
 * the paper's runs start each configuration from a fresh cache, Sec. 4.2).  Synchronises. */
int exmoe_cache_reset(exmoe_cache* cache, int layer);
/* Sticky device-side status of the cache's kernels (no paper counterpart): synchronises, returns EXMOE_OK or the last
 * EXMOE_ERR_BAD_EXPERT_ID / EXMOE_ERR_TIMEOUT raised on the device since the previous call, and clears it. */
int exmoe_status(exmoe_cache* cache);
/* Releases the library's own resources (events, copy stream, pinned staging, recorded graphs); the caller's buffers
 * stay the caller's (Sec. 3.3: slots and bank outlive individual requests).  Synchronises the device first. */
int exmoe_cache_destroy(exmoe_cache* cache);

/* Measurement hooks (the paper has no counterpart).  While enabled, every exmoe_moe_forward brackets
 * its kernels with CUDA events on the caller's stream, per kind: 0 = resolution + grouping,
 * 1 = gate/up GEMM + SwiGLU, 2 = down GEMM, 3 = combine, 4 = a wave's miss traffic (the fetch kernel on the
 * caller's stream, or the host-issued copies on the library's copy stream).  exmoe_profile_read synchronises and returns
 * the summed event time and the number of bracketed launches of one kind since the last enable.
 * Not for use during stream capture.
 * `on` bit 0 switches the event bracketing; bits 4-5, if non-zero, make later forwards launch ONLY
 * the kernels of that kind (1 gate/up, 2 down, 3 combine) so that one kernel can be timed alone, e.g.
 * in a CUDA-graph replay; the layer output is then meaningless.  exmoe_profile_enable(cache, 0)
 * restores normal operation. */
int exmoe_profile_enable(exmoe_cache* cache, int on);
int exmoe_profile_read(exmoe_cache* cache, int kind, double* total_ms, uint64_t* launches);
/* Evidence for Sec. 3.3's asynchronous miss copies: of the time the bracketed miss traffic (kind 4) was running since the
 * last enable, how much fell inside a bracketed GEMM interval (kinds 1 and 2) on the other stream.  Device timestamps of
 * the brackets' events; synchronises.  Both zero when nothing was bracketed. */
int exmoe_profile_overlap(exmoe_cache* cache, double* fetch_ms, double* fetch_during_gemm_ms);

/* Kernels launched by this library since it was loaded (all streams, all caches); measurement hook, no paper counterpart. */
uint64_t exmoe_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* EXMOE_H */
