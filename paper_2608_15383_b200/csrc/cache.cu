// Host side of the C ABI: slot caches (Section 3.3), the wave executor (Section 3.4), miss copies on a
// side stream ordered by events, and the test hooks.  All arithmetic of the path runs in kernels;
// this file only validates, carves the caller's workspace, launches and orders.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <new>
#include <map>
#include <vector>

#include "common.cuh"

namespace exmoe {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static int check_shape(const exmoe_shape* s) {
    if (!s) return EXMOE_ERR_ARG;
    if (s->group_size != kGroup) return EXMOE_ERR_SHAPE;
    if (s->d_model <= 0 || s->d_ff <= 0 || s->d_model % kGroup || s->d_ff % kGroup) return EXMOE_ERR_SHAPE;
    if (s->num_experts <= 0 || s->num_experts > 4096) return EXMOE_ERR_SHAPE;
    if (s->top_k <= 0 || s->top_k > s->num_experts) return EXMOE_ERR_SHAPE;
    return EXMOE_OK;
}

static size_t packed_bytes(const exmoe_shape& s) {
    return matrix_bytes(2 * s.d_ff, s.d_model) + matrix_bytes(s.d_model, s.d_ff);
}

struct Carve {                      // bump allocator over the caller's workspace (256-byte aligned pieces)
    uint8_t* base;
    size_t off = 0;
    template <typename T> T* take(size_t n) {
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += align_up(n * sizeof(T), 256);
        return p;
    }
};

constexpr int kEventRing = 64;
constexpr int kMaxKeys = 8192;      // ceil(E / wave_cap) * C: bounds the grouping kernels' shared memory

}  // namespace exmoe

using namespace exmoe;

struct exmoe_cache {
    exmoe_shape shape;
    int L, C, Cw, max_tokens, max_pairs, n_keys, max_waves;
    size_t bpe;                               // bytes per packed expert = slot stride
    std::vector<const uint8_t*> bank;
    std::vector<const uint8_t*> bank_dev;     // device-visible address of each bank (device-initiated miss path)
    int miss_path;                            // EXMOE_MISS_HOST_COPIES or EXMOE_MISS_DEVICE_FETCH
    uint8_t* slot_mem;
    int* d_status;
    std::vector<LayerState> state;
    PlanPtrs plan;
    PlanPtrs plan_pf;                         // resolution results of exmoe_cache_prefetch (its own copy: may overlap a forward)
    size_t plan_d2h_bytes;                    // header | wave_of | slot_of | misses, contiguous
    __nv_bfloat16* act;                       // [max_pairs, I] SwiGLU output, grouped row order
    float* y;                                 // [max_pairs, H] weighted expert outputs, pair order
    int* arrive;                              // fused-combine arrival counters of the small path
    size_t arrive_words;
    bool last_small;
    bool last_pair;
    int last_path;                            // EXMOE_PATH_* of the most recent forward
    int32_t* saved_ids;                       // ids of the last pairwise call (plan materialised on request)
    bool stream_ok;                           // the shape fits the streaming middle-regime kernels
    bool pair_ok, small_ok;                   // ... the per-pair kernels / the in-CTA-grouping kernels (shared memory)
    void* tc_scratch;                         // tile list of the tensor-core path
    __nv_bfloat16* xg;                        // [max_pairs, H] hidden rows in plan order (tensor-core path only)
    PrefillMaps tc_maps;                      // TMA descriptors of xg and act (a device array carved from the workspace)
    int32_t* h_plan;                          // pinned staging of the plan
    cudaStream_t copy_stream;
    cudaEvent_t ev_plan;
    cudaEvent_t ev_compute[kEventRing];       // completion of a wave's kernels (Section 3.4 step 5)
    cudaEvent_t ev_copy[kEventRing];          // completion of a wave's miss copies
    uint64_t seq;                             // last recorded compute event
    uint64_t copy_seq;
    std::vector<std::vector<uint64_t>> slot_last_seq;   // [L][C] compute event that last read the slot
    int last_layer;
    int last_T;
    bool prof_on;                             // per-kernel CUDA-event timing (exmoe_profile_*)
    int prof_only;                            // 0 = all kernels; 1..3 = launch only that kind (timing runs)
    std::vector<cudaEvent_t> prof_ev[5];      // begin/end pairs per kernel kind (4 = miss copies, copy stream)
    size_t prof_used[5];
    // exmoe_moe_forward_host: staging on both sides and one instantiated graph per (layer, T)
    uint8_t* d_stage;                         // device: hidden | ids | weights | out, each 256-byte aligned
    uint8_t* h_stage;                         // pinned host mirror of d_stage
    size_t stage_in_bytes, stage_out_off, stage_bytes;
    size_t last_host_h2d_bytes;               // bytes of the staged input copy of the last exmoe_moe_forward_host
    struct HostGraph {
        cudaGraphExec_t exec;
        bool last_small, last_pair;
        int last_path;
    };
    std::map<long long, HostGraph> host_graphs;
};

static void drop_host_graphs(exmoe_cache* c) {
    for (auto& kv : c->host_graphs) cudaGraphExecDestroy(kv.second.exec);
    c->host_graphs.clear();
}

enum { PROF_PLAN = 0, PROF_GATEUP = 1, PROF_DOWN = 2, PROF_COMBINE = 3, PROF_COPY = 4 };

// Brackets one launch (or launch group) with a pair of events on its own stream when profiling is on.
static void prof_mark(exmoe_cache* c, int kind, cudaStream_t st) {
    if (!c->prof_on) return;
    std::vector<cudaEvent_t>& v = c->prof_ev[kind];
    if (c->prof_used[kind] == v.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        v.push_back(e);
    }
    cudaEventRecord(v[c->prof_used[kind]++], st);
}
struct ProfScope {
    exmoe_cache* c;
    int kind;
    cudaStream_t st;
    ProfScope(exmoe_cache* c_, int kind_, cudaStream_t st_) : c(c_), kind(kind_), st(st_) { prof_mark(c, kind, st); }
    ~ProfScope() { prof_mark(c, kind, st); }
};

static void carve_workspace(exmoe_cache* c, uint8_t* ws, size_t* total) {
    const exmoe_shape& s = c->shape;
    const int E = s.num_experts, C = c->C;
    Carve k{ws};
    c->d_status = k.take<int>(64);
    c->state.resize(c->L);
    for (int l = 0; l < c->L; ++l) {
        c->state[l].expert_slot = k.take<int32_t>(E);
        c->state[l].slot_expert = k.take<int32_t>(C);
        c->state[l].slot_stamp = k.take<uint64_t>(C);
        c->state[l].tick = k.take<uint64_t>(1);
        c->state[l].stats = k.take<uint64_t>(6);
    }
    int32_t* p = k.take<int32_t>(HDR_WORDS + 5 * (size_t)E);
    c->plan.header = p;
    c->plan.wave_of = p ? p + HDR_WORDS : nullptr;
    c->plan.slot_of = p ? p + HDR_WORDS + E : nullptr;
    c->plan.misses = p ? p + HDR_WORDS + 2 * E : nullptr;
    c->plan_d2h_bytes = (HDR_WORDS + 5 * (size_t)E) * 4;
    c->plan.key_miss = k.take<int32_t>(c->n_keys);
    c->plan.n_keys = c->n_keys;
    int32_t* pf = k.take<int32_t>(HDR_WORDS + 5 * (size_t)E);
    c->plan_pf = PlanPtrs{};
    c->plan_pf.header = pf;
    c->plan_pf.wave_of = pf ? pf + HDR_WORDS : nullptr;
    c->plan_pf.slot_of = pf ? pf + HDR_WORDS + E : nullptr;
    c->plan_pf.misses = pf ? pf + HDR_WORDS + 2 * E : nullptr;
    c->plan_pf.key_miss = nullptr;                        // a prefetch runs no GEMM kernels
    c->plan_pf.n_keys = 0;
    c->plan.counts = k.take<int32_t>(c->n_keys);
    c->plan.offsets = k.take<int32_t>(c->n_keys + 1);
    c->plan.group_keys = k.take<int32_t>(c->n_keys);
    c->plan.wave_start = k.take<int32_t>(c->max_waves + 1);
    c->plan.perm = k.take<int32_t>(c->max_pairs);
    {
        const size_t chunks = ((size_t)c->max_pairs + 511) / 512;
        const size_t need = (size_t)c->n_keys * chunks, cap = (size_t)1 << 20;
        // reserve min(need, cap): monotone in the key space, so the size query (largest key space) bounds every create
        const size_t reserve = c->max_pairs <= 1024 ? 0 : (need < cap ? need : cap);
        int32_t* tab = reserve ? k.take<int32_t>(reserve) : nullptr;
        const bool usable = reserve && need <= cap;                       // larger key spaces keep the per-key scheme
        c->plan.chunk_table = usable ? tab : nullptr;
        c->plan.chunk_table_words = usable ? need : 0;
        c->plan.chunk_done = k.take<int32_t>(64);
    }
    c->act = k.take<__nv_bfloat16>((size_t)c->max_pairs * s.d_ff);
    c->y = k.take<float>((size_t)c->max_pairs * s.d_model);
    c->arrive_words = (size_t)(kSmallMaxPairs / s.top_k + 1) * (s.d_model / kPanelRows);
    c->arrive = k.take<int>(c->arrive_words);
    c->saved_ids = k.take<int32_t>(kPairMaxPairs);
    c->tc_scratch = k.take<uint8_t>(prefill_scratch_bytes(c->max_pairs, E));
    c->xg = (c->max_pairs > kSmallMaxPairs || !c->small_ok) ? k.take<__nv_bfloat16>((size_t)c->max_pairs * s.d_model) : nullptr;
    c->tc_maps.dev = c->xg ? k.take<uint8_t>(kPrefillMapBytes) : nullptr;
    {   // staging of the host-buffer entry point: hidden | ids | weights (one H2D copy), then out (one D2H copy)
        const size_t nb_h = align_up((size_t)c->max_tokens * s.d_model * 2, 256);
        const size_t nb_i = align_up((size_t)c->max_pairs * 4, 256);
        c->stage_in_bytes = nb_h + 2 * nb_i;
        c->stage_out_off = c->stage_in_bytes;
        c->stage_bytes = c->stage_in_bytes + nb_h;
        c->d_stage = k.take<uint8_t>(c->stage_bytes);
    }
    *total = k.off;
}

static int fill_dims(exmoe_cache* c, const exmoe_shape* shape, int num_layers, int num_slots, int max_tokens,
                     int wave_cap) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (num_layers <= 0 || max_tokens <= 0) return EXMOE_ERR_ARG;
    if (num_slots < shape->top_k || num_slots > shape->num_experts) return EXMOE_ERR_SHAPE;
    if (wave_cap < 0 || wave_cap > num_slots) return EXMOE_ERR_SHAPE;
    if ((long long)max_tokens * shape->top_k > (1ll << 30)) return EXMOE_ERR_ARG;
    c->shape = *shape;
    c->L = num_layers;
    c->C = num_slots;
    c->Cw = wave_cap ? wave_cap : num_slots;
    c->max_tokens = max_tokens;
    c->max_pairs = max_tokens * shape->top_k;
    c->max_waves = (shape->num_experts + c->Cw - 1) / c->Cw;
    c->n_keys = c->max_waves * c->C;
    if (c->n_keys > kMaxKeys) return EXMOE_ERR_SHAPE;
    c->bpe = packed_bytes(*shape);
    c->pair_ok = pair_path_fits(shape->d_model, shape->d_ff, shape->top_k);
    c->small_ok = small_path_fits(shape->d_model, shape->d_ff, c->C, kSmallMaxPairs);
    return EXMOE_OK;
}

static int reset_layer(exmoe_cache* c, int layer) {
    const int E = c->shape.num_experts, C = c->C;
    std::vector<int32_t> es(E, -1), se(C, -1);
    if (C == E)
        for (int e = 0; e < E; ++e) es[e] = se[e] = e;
    std::vector<uint64_t> zeros(C > 8 ? C : 8, 0);
    LayerState& st = c->state[layer];
    if (cudaMemcpy(st.expert_slot, es.data(), E * 4, cudaMemcpyHostToDevice) != cudaSuccess) return EXMOE_ERR_CUDA;
    if (cudaMemcpy(st.slot_expert, se.data(), C * 4, cudaMemcpyHostToDevice) != cudaSuccess) return EXMOE_ERR_CUDA;
    if (cudaMemcpy(st.slot_stamp, zeros.data(), C * 8, cudaMemcpyHostToDevice) != cudaSuccess) return EXMOE_ERR_CUDA;
    if (cudaMemcpy(st.tick, zeros.data(), 8, cudaMemcpyHostToDevice) != cudaSuccess) return EXMOE_ERR_CUDA;
    if (cudaMemcpy(st.stats, zeros.data(), 48, cudaMemcpyHostToDevice) != cudaSuccess) return EXMOE_ERR_CUDA;
    std::fill(c->slot_last_seq[layer].begin(), c->slot_last_seq[layer].end(), 0);
    return EXMOE_OK;
}

// Device-visible addresses of the host banks (the device-initiated miss path reads them over PCIe); false if a bank
// is not mapped into the device's address space or its mapped address is not 16-byte aligned.
static bool map_banks(exmoe_cache* c) {
    std::vector<const uint8_t*> devp;
    for (int l = 0; l < c->L; ++l) {
        void* d = nullptr;
        if (cudaHostGetDevicePointer(&d, const_cast<uint8_t*>(c->bank[l]), 0) != cudaSuccess || !d ||
            (reinterpret_cast<uintptr_t>(d) & 15)) {
            cudaGetLastError();
            return false;
        }
        devp.push_back(static_cast<const uint8_t*>(d));
    }
    c->bank_dev = devp;
    return true;
}

extern "C" {

const char* exmoe_strerror(int code) {
    switch (code) {
        case EXMOE_OK: return "ok";
        case EXMOE_ERR_ARG: return "invalid argument";
        case EXMOE_ERR_SHAPE: return "unsupported shape (dims must be multiples of 128, k <= C <= E)";
        case EXMOE_ERR_NOT_PINNED: return "host bank is not pinned host memory";
        case EXMOE_ERR_CUDA: return "CUDA runtime error";
        case EXMOE_ERR_NONFINITE: return "non-finite weight or scale overflow";
        case EXMOE_ERR_BAD_EXPERT_ID: return "expert id out of range";
        case EXMOE_ERR_TIMEOUT: return "bounded device wait expired";
        case EXMOE_ERR_STATE: return "call order";
        default: return "unknown error";
    }
}

uint64_t exmoe_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int exmoe_packed_bytes(const exmoe_shape* shape, size_t* bytes_per_expert) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!bytes_per_expert) return EXMOE_ERR_ARG;
    *bytes_per_expert = packed_bytes(*shape);
    return EXMOE_OK;
}

int exmoe_pack(const exmoe_shape* shape, const void* w_gate, const void* w_up, const void* w_down, void* packed_out,
               void* stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!w_gate || !w_up || !w_down || !packed_out) return EXMOE_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(packed_out) | reinterpret_cast<uintptr_t>(w_gate) |
         reinterpret_cast<uintptr_t>(w_up) | reinterpret_cast<uintptr_t>(w_down)) & 15)
        return EXMOE_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int* d_flag = pack_flag_word();
    if (!d_flag) return EXMOE_ERR_CUDA;
    int flag = 0;
    rc = EXMOE_OK;
    if (cudaMemsetAsync(d_flag, 0, sizeof(int), st) != cudaSuccess) rc = EXMOE_ERR_CUDA;
    if (!rc) rc = launch_pack(*shape, w_gate, w_up, w_down, packed_out, d_flag, st);
    if (!rc && cudaMemcpyAsync(&flag, d_flag, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) rc = EXMOE_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) rc = EXMOE_ERR_CUDA;
    if (!rc && flag) rc = EXMOE_ERR_NONFINITE;
    return rc;
}

int exmoe_cache_workspace_bytes(const exmoe_shape* shape, int num_layers, int num_slots, int max_tokens,
                                size_t* slot_bytes_total, size_t* workspace_bytes) {
    exmoe_cache tmp{};
    int rc = check_shape(shape);
    if (rc) return rc;
    int wc = 1;                                         // smallest wave_cap allowed = largest key space
    while (wc < num_slots && (long long)((shape->num_experts + wc - 1) / wc) * num_slots > kMaxKeys) ++wc;
    rc = fill_dims(&tmp, shape, num_layers, num_slots, max_tokens, wc);
    if (rc) return rc;
    if (!slot_bytes_total || !workspace_bytes) return EXMOE_ERR_ARG;
    *slot_bytes_total = (size_t)num_layers * num_slots * tmp.bpe;
    carve_workspace(&tmp, nullptr, workspace_bytes);
    return EXMOE_OK;
}

int exmoe_cache_create(exmoe_cache** out, const exmoe_shape* shape, int num_layers, int num_slots,
                       const void* const* host_bank, void* slot_mem, void* workspace, int max_tokens, int wave_cap) {
    if (!out || !host_bank || !slot_mem || !workspace) return EXMOE_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(slot_mem) | reinterpret_cast<uintptr_t>(workspace)) & 255) return EXMOE_ERR_ARG;
    exmoe_cache* c = new (std::nothrow) exmoe_cache{};
    if (!c) return EXMOE_ERR_ARG;
    int rc = fill_dims(c, shape, num_layers, num_slots, max_tokens, wave_cap);
    if (rc) { delete c; return rc; }
    for (int l = 0; l < num_layers; ++l) {
        cudaPointerAttributes attr{};
        if (!host_bank[l] || cudaPointerGetAttributes(&attr, host_bank[l]) != cudaSuccess ||
            attr.type != cudaMemoryTypeHost) {
            cudaGetLastError();
            delete c;
            return host_bank[l] ? EXMOE_ERR_NOT_PINNED : EXMOE_ERR_ARG;
        }
        c->bank.push_back(static_cast<const uint8_t*>(host_bank[l]));
    }
    c->slot_mem = static_cast<uint8_t*>(slot_mem);
    size_t total = 0;
    carve_workspace(c, static_cast<uint8_t*>(workspace), &total);
    c->slot_last_seq.assign(num_layers, std::vector<uint64_t>(num_slots, 0));
    c->last_layer = -1;
    c->last_T = 0;
    c->stream_ok = stream_supported(c->shape.d_model, c->shape.d_ff);
    c->miss_path = map_banks(c) ? EXMOE_MISS_DEVICE_FETCH : EXMOE_MISS_HOST_COPIES;
    bool ok = cudaMallocHost(&c->h_plan, c->plan_d2h_bytes) == cudaSuccess;
    ok = ok && cudaMallocHost(&c->h_stage, c->stage_bytes) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_plan, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < kEventRing && ok; ++i) {
        ok = ok && cudaEventCreateWithFlags(&c->ev_compute[i], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->ev_copy[i], cudaEventDisableTiming) == cudaSuccess;
    }
    ok = ok && cudaMemset(c->d_status, 0, 256) == cudaSuccess;
    ok = ok && cudaMemset(c->plan.header, 0, c->plan_d2h_bytes) == cudaSuccess;
    ok = ok && cudaMemset(c->plan_pf.header, 0, c->plan_d2h_bytes) == cudaSuccess;
    ok = ok && cudaMemset(c->arrive, 0, c->arrive_words * 4) == cudaSuccess;
    ok = ok && cudaMemset(c->plan.chunk_done, 0, 256) == cudaSuccess;
    for (int l = 0; l < num_layers && ok; ++l) ok = reset_layer(c, l) == EXMOE_OK;
    if (ok && c->xg) ok = prefill_setup(&c->tc_maps, c->xg, c->act, c->max_pairs, c->shape.d_model, c->shape.d_ff) == EXMOE_OK;
    if (ok && c->C == c->shape.num_experts) {            // full residency: preload, slot = expert id
        for (int l = 0; l < num_layers && ok; ++l)
            ok = cudaMemcpy(c->slot_mem + (size_t)l * c->C * c->bpe, c->bank[l], (size_t)c->C * c->bpe,
                            cudaMemcpyHostToDevice) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        exmoe_cache_destroy(c);
        return EXMOE_ERR_CUDA;
    }
    *out = c;
    return EXMOE_OK;
}

int exmoe_moe_forward(exmoe_cache* c, int layer, const void* hidden, const int32_t* topk_ids,
                      const float* topk_weights, int T, void* out, void* stream) {
    if (!c || layer < 0 || layer >= c->L || T < 0 || T > c->max_tokens) return EXMOE_ERR_ARG;
    if (T == 0) return EXMOE_OK;
    if (!hidden || !topk_ids || !topk_weights || !out) return EXMOE_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden) | reinterpret_cast<uintptr_t>(out)) & 15) return EXMOE_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const exmoe_shape& s = c->shape;
    const int E = s.num_experts, C = c->C, k = s.top_k, P = T * k;
    const bool identity = (C == E);
    const bool dev_fetch = !identity && c->miss_path == EXMOE_MISS_DEVICE_FETCH;   // no host wait, no host-issued copies
    c->last_layer = layer;
    c->last_T = T;

    const bool small = (P <= kSmallMaxPairs && C <= kSmallMaxSlots && c->small_ok);   // decode: grouping fused into the GEMM kernels
    c->last_small = small;
    if (!identity) {
        ProfScope ps(c, PROF_PLAN, st);
        launch_resolve(s, C, c->Cw, c->bpe, topk_ids, P, c->state[layer], c->plan, c->d_status, st);
        if (!dev_fetch) {
            if (cudaMemcpyAsync(c->h_plan, c->plan.header, c->plan_d2h_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
                return EXMOE_ERR_CUDA;
            if (cudaEventRecord(c->ev_plan, st) != cudaSuccess) return EXMOE_ERR_CUDA;
        }
    }
    // timing runs that launch one kernel kind reuse the plan, grouped rows and tile list of the previous full call
    const bool build_plan = (c->prof_only == 0);
    if (!small && build_plan) {
        ProfScope ps(c, PROF_PLAN, st);
        launch_group(s, C, c->n_keys, c->max_waves, identity, topk_ids, P, c->plan, c->d_status, st);
    }

    int n_waves = 1;
    const int32_t *h_wave_of = nullptr, *h_slot_of = nullptr, *h_miss = nullptr;
    int n_miss = 0;
    if (dev_fetch) {
        // The host does not learn the plan.  A call activates at most min(P, E) experts and a wave holds up to
        // wave_cap of them, so this many waves always suffice; a wave that turns out empty costs its launches only
        // (every kernel takes its group count from the device plan and finds nothing to do).
        const int act_max = P < E ? P : E;
        n_waves = (act_max + c->Cw - 1) / c->Cw;
        if (n_waves > c->max_waves) n_waves = c->max_waves;
        if (n_waves < 1) n_waves = 1;
    } else if (!identity) {
        if (cudaEventSynchronize(c->ev_plan) != cudaSuccess) return EXMOE_ERR_CUDA;   // the one batched id transfer
        n_waves = c->h_plan[HDR_N_WAVES];
        n_miss = c->h_plan[HDR_N_MISSES];
        h_wave_of = c->h_plan + HDR_WORDS;
        h_slot_of = h_wave_of + E;
        h_miss = h_slot_of + E;
    }

    GemmArgs a{};
    a.slots = c->slot_mem + (size_t)layer * C * c->bpe;
    a.slot_stride = c->bpe;
    a.counts = c->plan.counts;
    a.offsets = c->plan.offsets;
    a.group_keys = c->plan.group_keys;
    a.perm = c->plan.perm;
    a.key_miss = c->plan.key_miss;
    a.group_filter = 0;
    a.direct_keys = (C == E && c->n_keys <= 128) ? c->n_keys : 0;
    a.num_slots = C;
    a.top_k = k;
    a.H = s.d_model;
    a.I = s.d_ff;

    bool tiles_fused = false;
    const bool pairwise = small && P <= kPairMaxPairs && n_waves == 1 && c->pair_ok;
    c->last_pair = pairwise;
    const bool use_stream = !small && c->stream_ok && P <= kStreamMaxPairs;
    const bool small_n = P <= kPrefillSmallNMaxPairs;      // tensor-core path: which kernel shape
    c->last_path = pairwise ? EXMOE_PATH_PAIR : small ? EXMOE_PATH_SMALL : use_stream ? EXMOE_PATH_STREAM
                   : small_n ? EXMOE_PATH_TENSOR_SMALL_N : EXMOE_PATH_TENSOR;
    if (!small && build_plan && !use_stream) {
        ProfScope ps(c, PROF_PLAN, st);                  // hidden rows in plan order, once for all waves
        tiles_fused = (n_waves == 1);                    // one wave: its tile list comes out of the same launch
        launch_gather_rows((const __nv_bfloat16*)hidden, c->plan.perm, c->plan.offsets + c->n_keys, P, k, s.d_model,
                           c->xg, tiles_fused ? &a : nullptr, c->plan.wave_start, c->tc_scratch, small_n, st);
    }
    if (small && n_waves == 0)                           // no valid id at all: the output is zero
        cudaMemsetAsync(out, 0, (size_t)T * s.d_model * 2, st);
    int mi = 0;
    for (int w = 0; w < n_waves; ++w) {
        int groups = identity ? (E < P ? E : P) : 0;
        bool split = false;                              // the wave's kernels run twice: resident groups, then fetched ones
        if (dev_fetch) {
#ifndef EXMOE_NO_FETCH_OVERLAP
            split = use_stream && !c->prof_only;
#endif
            if (split) {
                // Sec. 3.3's asynchronous miss copy, Sec. 3.4 steps 3-5: the wave's fetch kernel runs on the library's side
                // stream, behind everything that may still read the slots it overwrites (resolution and grouping for the
                // first wave, the previous wave's kernels after that); meanwhile the wave's kernels run over the groups
                // whose experts were resident (a miss only evicts slots the wave does not use), then wait for the fetch
                // and run over the fetched groups.  Ordered by events in both directions: no kernel polls another.
                cudaEvent_t fork = c->ev_compute[(++c->seq) % kEventRing];
                cudaEventRecord(fork, st);
                cudaStreamWaitEvent(c->copy_stream, fork, 0);
                {
                    ProfScope ps(c, PROF_COPY, c->copy_stream);
                    launch_fetch_misses(c->plan, w, c->bank_dev[layer], const_cast<uint8_t*>(a.slots), c->bpe, E, C, c->copy_stream,
                                        false, /*follows_resolve=*/false);
                }
                cudaEventRecord(c->ev_copy[(++c->copy_seq) % kEventRing], c->copy_stream);
            } else {
                ProfScope ps(c, PROF_COPY, st);
                launch_fetch_misses(c->plan, w, c->bank_dev[layer], const_cast<uint8_t*>(a.slots), c->bpe, E, C, st);
            }
            groups = c->Cw < P ? c->Cw : P;              // upper bound of the wave's groups (sizes the grids only)
            if (groups > E) groups = E;
        } else if (!identity) {
            bool copied = false;
            const bool wave_has_miss = mi < n_miss && h_miss[3 * mi + 2] == w;
            if (wave_has_miss) prof_mark(c, PROF_COPY, c->copy_stream);       // begin of the wave's copies
            for (; mi < n_miss && h_miss[3 * mi + 2] == w; ++mi) {
                const int e = h_miss[3 * mi], v = h_miss[3 * mi + 1];
                // the wave that last read the slot; once the ring has wrapped its entry belongs to a later wave, so the
                // most recent compute event stands in (all forwards of a cache share one stream order: see exmoe.h)
                const uint64_t last = c->slot_last_seq[layer][v];
                if (last) cudaStreamWaitEvent(c->copy_stream, c->ev_compute[(c->seq - last >= kEventRing ? c->seq : last) % kEventRing], 0);
                if (cudaMemcpyAsync(const_cast<uint8_t*>(a.slots) + (size_t)v * c->bpe, c->bank[layer] + (size_t)e * c->bpe,
                                    c->bpe, cudaMemcpyHostToDevice, c->copy_stream) != cudaSuccess)
                    return EXMOE_ERR_CUDA;
                copied = true;
            }
            if (copied) prof_mark(c, PROF_COPY, c->copy_stream);              // end of the wave's copies
            if (copied) {
                cudaEvent_t ev = c->ev_copy[(++c->copy_seq) % kEventRing];
                cudaEventRecord(ev, c->copy_stream);
                cudaStreamWaitEvent(st, ev, 0);
            }
            for (int e = 0; e < E; ++e) groups += (h_wave_of[e] == w);
        }
        a.wave_start = c->plan.wave_start + w;
        if (small) {
            SmallWave sw{};
            sw.ids = topk_ids;
            sw.wave_of = identity ? nullptr : c->plan.wave_of;
            sw.slot_of = identity ? nullptr : c->plan.slot_of;
            sw.n_pairs = P;
            sw.E = E;
            sw.wave = w;
            sw.plan = c->plan;
            sw.status = c->d_status;
            sw.arrive = c->arrive;
            sw.hidden = (const __nv_bfloat16*)hidden;
            sw.act = c->act;
            sw.topk_w = topk_weights;
            sw.y = c->y;
            sw.out = (__nv_bfloat16*)out;
            sw.max_rows = T;
            sw.max_groups = groups;
            sw.pairwise = pairwise;
            sw.saved_ids = c->saved_ids;
            if (pairwise && !c->prof_only && !c->prof_on) {
                launch_small_wave(a, sw, st, true, true);
            } else {
                if (!c->prof_only || c->prof_only == PROF_GATEUP) {
                    ProfScope ps(c, PROF_GATEUP, st);
                    launch_small_wave(a, sw, st, true, false);
                }
                if (!c->prof_only || c->prof_only == PROF_DOWN) {
                    ProfScope ps(c, PROF_DOWN, st);
                    launch_small_wave(a, sw, st, false, true);
                }
            }
        } else if (use_stream) {
            // a few to a few dozen rows per expert: bulk-copy weight ring + register dequantisation, pair buffer + combine
            if (split) {
                a.group_filter = 1;
                {
                    ProfScope ps(c, PROF_GATEUP, st);
                    launch_stream_wave(a, (const __nv_bfloat16*)hidden, c->act, topk_weights, c->y, c->d_status, groups, true, true, st);
                }
                cudaStreamWaitEvent(st, c->ev_copy[c->copy_seq % kEventRing], 0);     // the wave's fetched experts are in their slots
                a.group_filter = 2;
                {
                    ProfScope ps(c, PROF_GATEUP, st);
                    launch_stream_wave(a, (const __nv_bfloat16*)hidden, c->act, topk_weights, c->y, c->d_status, groups, true, true, st);
                }
                a.group_filter = 0;
            } else if (!c->prof_only) {
                ProfScope ps(c, PROF_GATEUP, st);    // both kernels: the down kernel is a programmatic dependent
                launch_stream_wave(a, (const __nv_bfloat16*)hidden, c->act, topk_weights, c->y, c->d_status, groups, true, true,
                                   st);
            } else if (c->prof_only == PROF_GATEUP || c->prof_only == PROF_DOWN) {
                ProfScope ps(c, c->prof_only, st);
                launch_stream_wave(a, (const __nv_bfloat16*)hidden, c->act, topk_weights, c->y, c->d_status, groups,
                                   c->prof_only == PROF_GATEUP, c->prof_only == PROF_DOWN, st);
            }
        } else {
            // many rows per expert: dense contraction on the tensor cores (tcgen05 / TMEM)
            if (build_plan && !tiles_fused)
                launch_prefill_wave(a, a.wave_start, c->tc_scratch, c->d_status, &c->tc_maps, c->act, topk_weights, c->y, 4, small_n, st);
            if (!c->prof_only || c->prof_only == PROF_GATEUP) {
                ProfScope ps(c, PROF_GATEUP, st);
                launch_prefill_wave(a, a.wave_start, c->tc_scratch, c->d_status, &c->tc_maps, c->act, topk_weights, c->y, 1,
                                    small_n, st);
            }
            if (!c->prof_only || c->prof_only == PROF_DOWN) {
                ProfScope ps(c, PROF_DOWN, st);
                launch_prefill_wave(a, a.wave_start, c->tc_scratch, c->d_status, &c->tc_maps, c->act, topk_weights, c->y, 2,
                                    small_n, st);
            }
        }
        if (!identity && !dev_fetch) {
            ++c->seq;
            cudaEventRecord(c->ev_compute[c->seq % kEventRing], st);                  // completion event of the wave
            for (int e = 0; e < E; ++e)
                if (h_wave_of[e] == w) c->slot_last_seq[layer][h_slot_of[e]] = c->seq;
        }
    }
    if (!small && (!c->prof_only || c->prof_only == PROF_COMBINE)) {
        ProfScope ps(c, PROF_COMBINE, st);
        launch_combine(c->y, topk_ids, E, T, k, s.d_model, (__nv_bfloat16*)out, st);
    }
    return cudaGetLastError() == cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int exmoe_cache_set_miss_path(exmoe_cache* c, int mode) {
    if (!c || (mode != EXMOE_MISS_HOST_COPIES && mode != EXMOE_MISS_DEVICE_FETCH)) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;     // no wave of the other mode is in flight
    if (mode == EXMOE_MISS_DEVICE_FETCH && !map_banks(c)) return EXMOE_ERR_NOT_PINNED;
    for (auto& v : c->slot_last_seq) std::fill(v.begin(), v.end(), 0);       // everything earlier has completed
    drop_host_graphs(c);                                                     // they hold the other mode's launch sequence
    c->miss_path = mode;
    return EXMOE_OK;
}

int exmoe_moe_forward_host(exmoe_cache* c, int layer, const void* hidden_host, const int32_t* ids_host,
                           const float* weights_host, int T, void* out_host, void* stream) {
    if (!c || layer < 0 || layer >= c->L || T < 0 || T > c->max_tokens) return EXMOE_ERR_ARG;
    if (T == 0) return EXMOE_OK;
    if (!hidden_host || !ids_host || !weights_host || !out_host) return EXMOE_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const exmoe_shape& s = c->shape;
    const size_t nb_h = (size_t)T * s.d_model * 2, nb_i = (size_t)T * s.top_k * 4;
    // hidden | ids | weights back to back (16-byte aligned pieces), so that the one H2D copy moves what this call needs
    // and not what max_tokens would; the recorded graphs are keyed by T, so T-dependent offsets are safe
    const size_t off_i = align_up(nb_h, 16);
    const size_t off_w = off_i + align_up(nb_i, 16);
    void* d_h = c->d_stage;
    int32_t* d_i = reinterpret_cast<int32_t*>(c->d_stage + off_i);
    float* d_w = reinterpret_cast<float*>(c->d_stage + off_w);
    // Small results are written by the last kernel straight into the pinned staging buffer (mapped into the device's
    // address space; posted writes over the host link), which saves the copy node after the layer.
    const bool out_direct = nb_h <= ((size_t)64 << 10);
    void* d_o = out_direct ? static_cast<void*>(c->h_stage + c->stage_out_off) : static_cast<void*>(c->d_stage + c->stage_out_off);
    // Large calls whose tensors are page-locked already skip the staging copies (8 MB each way at 2048 tokens would
    // cost more than the layer): the device copies read and write the caller's memory, as plain launches.
    if (nb_h >= ((size_t)256 << 10)) {
        bool pinned = true;
        const void* ptrs[4] = {hidden_host, ids_host, weights_host, out_host};
        for (int i = 0; i < 4 && pinned; ++i) {
            cudaPointerAttributes attr{};
            pinned = cudaPointerGetAttributes(&attr, ptrs[i]) == cudaSuccess && attr.type == cudaMemoryTypeHost;
        }
        cudaGetLastError();
        if (pinned) {
            c->last_host_h2d_bytes = nb_h + 2 * nb_i;
            bool ok = cudaMemcpyAsync(d_h, hidden_host, nb_h, cudaMemcpyHostToDevice, st) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(d_i, ids_host, nb_i, cudaMemcpyHostToDevice, st) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(d_w, weights_host, nb_i, cudaMemcpyHostToDevice, st) == cudaSuccess;
            int rc = ok ? exmoe_moe_forward(c, layer, d_h, d_i, d_w, T, d_o, st) : EXMOE_ERR_CUDA;
            if (!rc && cudaMemcpyAsync(out_host, d_o, nb_h, cudaMemcpyDeviceToHost, st) != cudaSuccess) rc = EXMOE_ERR_CUDA;
            if (cudaStreamSynchronize(st) != cudaSuccess) rc = rc ? rc : EXMOE_ERR_CUDA;
            return rc;
        }
    }
    std::memcpy(c->h_stage, hidden_host, nb_h);
    std::memcpy(c->h_stage + off_i, ids_host, nb_i);
    std::memcpy(c->h_stage + off_w, weights_host, nb_i);
    const size_t in_bytes = off_w + nb_i;                                 // one copy covers the three inputs
    c->last_host_h2d_bytes = in_bytes;
    auto enqueue = [&]() -> int {
        if (cudaMemcpyAsync(c->d_stage, c->h_stage, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return EXMOE_ERR_CUDA;
        const int rc = exmoe_moe_forward(c, layer, d_h, d_i, d_w, T, d_o, st);
        if (rc) return rc;
        if (!out_direct &&
            cudaMemcpyAsync(c->h_stage + c->stage_out_off, d_o, nb_h, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return EXMOE_ERR_CUDA;
        return EXMOE_OK;
    };
    // The launch sequence of a call is fixed when no host wait sits inside it (all experts resident, or the
    // device-initiated miss path): it is then captured once per (layer, T) and replayed, one graph launch per call.
    // Only for the tiny-batch path: rotating over 16 layer banks, one token per call, the replay gives 30.4 k calls/s
    // against 28.6 k with plain launches; at 16 tokens (grouping, two GEMM kernels, combine) plain launches win,
    // 207 k against 197 k tokens/s, and the larger the call the less the launches matter.
    const bool fixed = (c->C == s.num_experts || c->miss_path == EXMOE_MISS_DEVICE_FETCH) && !c->prof_on && !c->prof_only &&
                       T * s.top_k <= kSmallMaxPairs;
    const long long key = (long long)layer * ((long long)c->max_tokens + 1) + T;
    int rc = EXMOE_OK;
    auto it = fixed ? c->host_graphs.find(key) : c->host_graphs.end();
    if (it != c->host_graphs.end()) {
        c->last_layer = layer;
        c->last_T = T;
        c->last_small = it->second.last_small;
        c->last_pair = it->second.last_pair;
        c->last_path = it->second.last_path;
        if (cudaGraphLaunch(it->second.exec, st) != cudaSuccess) rc = EXMOE_ERR_CUDA;
    } else {
        rc = enqueue();                                                   // this call runs as plain launches
    }
    if (cudaStreamSynchronize(st) != cudaSuccess) rc = rc ? rc : EXMOE_ERR_CUDA;
    if (!rc) std::memcpy(out_host, c->h_stage + c->stage_out_off, nb_h);
    if (!rc && fixed && it == c->host_graphs.end() && c->host_graphs.size() < 256) {
        // ... and the same sequence is recorded for the next call of this (layer, T); recording launches nothing
        cudaGraph_t g = nullptr;
        cudaGraphExec_t exec = nullptr;
        bool ok = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
        if (ok) {
            const int crc = enqueue();
            ok = cudaStreamEndCapture(st, &g) == cudaSuccess && crc == EXMOE_OK && g;
        }
        ok = ok && cudaGraphInstantiate(&exec, g, 0) == cudaSuccess;
        if (g) cudaGraphDestroy(g);
        if (ok) c->host_graphs[key] = exmoe_cache::HostGraph{exec, c->last_small, c->last_pair, c->last_path};
        else cudaGetLastError();                                          // stay on plain launches for this key
    }
    return rc;
}

int exmoe_cache_prefetch(exmoe_cache* c, int layer, const int32_t* expert_ids, int n_ids, void* stream) {
    if (!c || layer < 0 || layer >= c->L || n_ids < 0 || n_ids > c->max_pairs) return EXMOE_ERR_ARG;
    if (n_ids == 0 || c->C == c->shape.num_experts) return EXMOE_OK;          // nothing to bring in
    if (!expert_ids) return EXMOE_ERR_ARG;
    if (c->miss_path != EXMOE_MISS_DEVICE_FETCH) return EXMOE_ERR_STATE;
    cudaStream_t st = (cudaStream_t)stream;
    const int E = c->shape.num_experts;
    launch_resolve(c->shape, c->C, c->Cw, c->bpe, expert_ids, n_ids, c->state[layer], c->plan_pf, c->d_status, st);
    const int act_max = n_ids < E ? n_ids : E;
    int n_waves = (act_max + c->Cw - 1) / c->Cw;
    if (n_waves > c->max_waves) n_waves = c->max_waves;
    for (int w = 0; w < n_waves; ++w)
        launch_fetch_misses(c->plan_pf, w, c->bank_dev[layer], c->slot_mem + (size_t)layer * c->C * c->bpe, c->bpe, E, c->C, st,
                            /*small_grid=*/true);
    return cudaGetLastError() == cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int exmoe_cache_get_state(exmoe_cache* c, int layer, int32_t* expert_slot, int32_t* slot_expert, uint64_t* slot_stamp,
                          uint64_t* tick) {
    if (!c || layer < 0 || layer >= c->L) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    const LayerState& st = c->state[layer];
    bool ok = true;
    if (expert_slot) ok = ok && cudaMemcpy(expert_slot, st.expert_slot, c->shape.num_experts * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (slot_expert) ok = ok && cudaMemcpy(slot_expert, st.slot_expert, c->C * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (slot_stamp) ok = ok && cudaMemcpy(slot_stamp, st.slot_stamp, c->C * 8, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (tick) ok = ok && cudaMemcpy(tick, st.tick, 8, cudaMemcpyDeviceToHost) == cudaSuccess;
    return ok ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int exmoe_debug_last_plan(exmoe_cache* c, int layer, int32_t* n_active, int32_t* n_waves, int32_t* n_misses,
                          int32_t* wave_of, int32_t* slot_of, int32_t* counts, int32_t* offsets, int32_t* perm,
                          int32_t* misses) {
    if (!c || layer < 0 || layer >= c->L) return EXMOE_ERR_ARG;
    if (layer != c->last_layer) return EXMOE_ERR_STATE;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    const int E = c->shape.num_experts;
    if (c->last_pair) {
        // the pairwise path never groups: run the grouping kernel now on the ids it kept
        launch_group(c->shape, c->C, c->n_keys, c->max_waves, c->C == E, c->saved_ids, c->last_T * c->shape.top_k,
                     c->plan, c->d_status, nullptr);
        if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
        c->last_pair = false;
        c->last_small = false;
    }
    std::vector<int32_t> hdr(HDR_WORDS + 5 * (size_t)E);
    bool ok = cudaMemcpy(hdr.data(), c->plan.header, hdr.size() * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    std::vector<int32_t> cnt(c->n_keys);
    ok = ok && cudaMemcpy(cnt.data(), c->plan.counts, cnt.size() * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (!ok) return EXMOE_ERR_CUDA;
    std::vector<int32_t> off(c->n_keys + 1);
    ok = cudaMemcpy(off.data(), c->plan.offsets, off.size() * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (!ok) return EXMOE_ERR_CUDA;
    if (c->last_small) {                                 // each wave's kernel published its own part only
        const int first = hdr[HDR_N_WAVES] * c->C;
        int total = 0;
        for (int i = 0; i < first; ++i) total += cnt[i];
        for (int i = first; i < c->n_keys; ++i) cnt[i] = 0;
        for (int i = first; i <= c->n_keys; ++i) off[i] = total;
    }
    if (n_active) *n_active = hdr[HDR_N_ACTIVE];
    if (n_waves) *n_waves = hdr[HDR_N_WAVES];
    if (n_misses) *n_misses = hdr[HDR_N_MISSES];
    const bool identity = (c->C == E);
    if (wave_of)
        for (int e = 0; e < E; ++e) wave_of[e] = identity ? (cnt[e] > 0 ? 0 : -1) : hdr[HDR_WORDS + e];
    if (slot_of)
        for (int e = 0; e < E; ++e) slot_of[e] = identity ? (cnt[e] > 0 ? e : -1) : hdr[HDR_WORDS + E + e];
    if (misses) std::memcpy(misses, hdr.data() + HDR_WORDS + 2 * E, 3 * (size_t)E * 4);
    if (counts) std::memcpy(counts, cnt.data(), cnt.size() * 4);
    if (offsets) std::memcpy(offsets, off.data(), off.size() * 4);
    if (perm) ok = ok && cudaMemcpy(perm, c->plan.perm, (size_t)c->last_T * c->shape.top_k * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    return ok ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int exmoe_debug_last_path(exmoe_cache* c) {
    if (!c) return EXMOE_ERR_ARG;
    if (c->last_layer < 0) return EXMOE_ERR_STATE;
    return c->last_path;
}

int exmoe_debug_last_host_copy_bytes(exmoe_cache* c, size_t* h2d_bytes) {
    if (!c || !h2d_bytes) return EXMOE_ERR_ARG;
    *h2d_bytes = c->last_host_h2d_bytes;
    return EXMOE_OK;
}

int exmoe_debug_read_slot(exmoe_cache* c, int layer, int slot, void* host_out) {
    if (!c || layer < 0 || layer >= c->L || slot < 0 || slot >= c->C || !host_out) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    return cudaMemcpy(host_out, c->slot_mem + ((size_t)layer * c->C + slot) * c->bpe, c->bpe, cudaMemcpyDeviceToHost) ==
                   cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int exmoe_cache_stats(exmoe_cache* c, int layer, exmoe_stats* out) {
    if (!c || layer < 0 || layer >= c->L || !out) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    uint64_t v[6];
    if (cudaMemcpy(v, c->state[layer].stats, 48, cudaMemcpyDeviceToHost) != cudaSuccess) return EXMOE_ERR_CUDA;
    out->lookups = v[0]; out->hits = v[1]; out->misses = v[2]; out->waves = v[3]; out->h2d_bytes = v[4]; out->forwards = v[5];
    return EXMOE_OK;
}

int exmoe_cache_reset(exmoe_cache* c, int layer) {
    if (!c || layer < 0 || layer >= c->L) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    return reset_layer(c, layer);
}

int exmoe_status(exmoe_cache* c) {
    if (!c) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, c->d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return EXMOE_ERR_CUDA;
    if (v && cudaMemset(c->d_status, 0, 4) != cudaSuccess) return EXMOE_ERR_CUDA;
    return v;
}

int exmoe_profile_enable(exmoe_cache* c, int on) {
    if (!c) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    c->prof_on = (on & 1) != 0;
    c->prof_only = (on >> 4) & 3;
    for (int k = 0; k < 5; ++k) c->prof_used[k] = 0;
    return EXMOE_OK;
}

int exmoe_profile_read(exmoe_cache* c, int kind, double* total_ms, uint64_t* launches) {
    if (!c || kind < 0 || kind > 4 || !total_ms || !launches) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    double sum = 0.0;
    const size_t n = c->prof_used[kind] / 2;
    for (size_t i = 0; i < n; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, c->prof_ev[kind][2 * i], c->prof_ev[kind][2 * i + 1]) != cudaSuccess)
            return EXMOE_ERR_CUDA;
        sum += ms;
    }
    *total_ms = sum;
    *launches = n;
    return EXMOE_OK;
}

int exmoe_profile_overlap(exmoe_cache* c, double* fetch_ms, double* fetch_during_gemm_ms) {
    if (!c || !fetch_ms || !fetch_during_gemm_ms) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    // device timestamps of every bracketed interval, relative to the first GEMM bracket (all events are on one device)
    auto intervals = [&](int kind, cudaEvent_t ref, std::vector<std::pair<double, double>>& out) -> bool {
        for (size_t i = 0; i + 1 < c->prof_used[kind]; i += 2) {
            float t0 = 0.f, t1 = 0.f;
            if (cudaEventElapsedTime(&t0, ref, c->prof_ev[kind][i]) != cudaSuccess ||
                cudaEventElapsedTime(&t1, ref, c->prof_ev[kind][i + 1]) != cudaSuccess)
                return false;
            out.emplace_back((double)t0, (double)t1);
        }
        return true;
    };
    *fetch_ms = *fetch_during_gemm_ms = 0.0;
    if (c->prof_used[PROF_COPY] < 2 || c->prof_used[PROF_GATEUP] < 2) return EXMOE_OK;
    cudaEvent_t ref = c->prof_ev[PROF_GATEUP][0];
    std::vector<std::pair<double, double>> f, g;
    if (!intervals(PROF_COPY, ref, f) || !intervals(PROF_GATEUP, ref, g) || !intervals(PROF_DOWN, ref, g)) {
        cudaGetLastError();
        return EXMOE_ERR_CUDA;
    }
    for (const auto& fi : f) {
        *fetch_ms += fi.second - fi.first;
        for (const auto& gi : g) {
            const double lo = std::max(fi.first, gi.first), hi = std::min(fi.second, gi.second);
            if (hi > lo) *fetch_during_gemm_ms += hi - lo;
        }
    }
    return EXMOE_OK;
}

int exmoe_debug_wait_timeout(exmoe_cache* c, long long budget_cycles, int* gave_up) {
    if (!c || !gave_up || budget_cycles <= 0 || budget_cycles > 4000000000ll) return EXMOE_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    int* d_result = c->d_status + 8;                       // spare word of the status block
    launch_wait_selftest(c->d_status, budget_cycles, d_result, nullptr);
    if (cudaDeviceSynchronize() != cudaSuccess) return EXMOE_ERR_CUDA;
    return cudaMemcpy(gave_up, d_result, 4, cudaMemcpyDeviceToHost) == cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}

int exmoe_cache_destroy(exmoe_cache* c) {
    if (!c) return EXMOE_ERR_ARG;
    cudaDeviceSynchronize();
    for (int k = 0; k < 5; ++k)
        for (cudaEvent_t e : c->prof_ev[k]) cudaEventDestroy(e);
    drop_host_graphs(c);
    if (c->h_plan) cudaFreeHost(c->h_plan);
    if (c->h_stage) cudaFreeHost(c->h_stage);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    if (c->ev_plan) cudaEventDestroy(c->ev_plan);
    for (int i = 0; i < kEventRing; ++i) {
        if (c->ev_compute[i]) cudaEventDestroy(c->ev_compute[i]);
        if (c->ev_copy[i]) cudaEventDestroy(c->ev_copy[i]);
    }
    delete c;
    return EXMOE_OK;
}

}  // extern "C"
