// Fused router (Eq. 1 of the paper, Section 3.1): z_t = W_r h_t (+ optional per-expert bias), softmax over all
// E experts, the k largest (ties to the lower expert id), mixture weights = the selected probabilities, not
// renormalised (Section 3.4).  It produces exmoe_moe_forward's `topk_ids` / `topk_weights` on the device, so a
// whole stack step can be captured in one CUDA graph without host-side routing.
//
// One CTA per token.  The router matrix (E x H BF16, 256 KB for OLMoE) is shared by all tokens and stays in L2;
// the token's hidden row is staged in shared memory once; warp w computes the logits of experts w, w+8, ...
// with 128-bit loads, binary32 accumulation in a fixed order (lane-strided partial sums, then a shuffle tree).
// Warp 0 then does the softmax (expf, binary32) and k rounds of a warp-wide arg-max whose comparison orders
// equal probabilities by ascending id.  Latency-bound and small next to the expert GEMMs.
#include "common.cuh"

namespace exmoe {

namespace {

constexpr int kRouteThreads = 256;

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b) {
    const uint32_t x[4] = {a.x, a.y, a.z, a.w}, y[4] = {b.x, b.y, b.z, b.w};
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        s = fmaf(__uint_as_float(x[i] << 16), __uint_as_float(y[i] << 16), s);
        s = fmaf(__uint_as_float(x[i] & 0xffff0000u), __uint_as_float(y[i] & 0xffff0000u), s);
    }
    return s;
}

__global__ void __launch_bounds__(kRouteThreads)
route_kernel(const __nv_bfloat16* __restrict__ hidden, const __nv_bfloat16* __restrict__ w_router,
             const float* __restrict__ bias, int H, int E, int k, int32_t* __restrict__ ids_out,
             float* __restrict__ w_out) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);                       // [H / 8] the token's hidden row
    float* prob = reinterpret_cast<float*>(smem + (size_t)H * 2);      // [E] logits, then probabilities
    const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunks = H / 8;
    const uint4* xrow = reinterpret_cast<const uint4*>(hidden + (size_t)t * H);
    for (int i = tid; i < chunks; i += kRouteThreads) xs[i] = xrow[i];
    __syncthreads();
    for (int e = warp; e < E; e += kRouteThreads / 32) {
        const uint4* wrow = reinterpret_cast<const uint4*>(w_router + (size_t)e * H);
        float s = 0.f;
        for (int i = lane; i < chunks; i += 32) s += dot8(wrow[i], xs[i]);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
        if (lane == 0) prob[e] = s + (bias ? bias[e] : 0.f);
    }
    __syncthreads();
    if (warp != 0) return;
    float mx = -INFINITY;
    for (int e = lane; e < E; e += 32) mx = fmaxf(mx, prob[e]);
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, m));
    float sum = 0.f;
    for (int e = lane; e < E; e += 32) {
        const float v = expf(prob[e] - mx);
        prob[e] = v;
        sum += v;
    }
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
    __syncwarp();
    const float inv = 1.f / sum;
    for (int j = 0; j < k; ++j) {
        // arg-max over the experts not yet taken (taken ones are marked negative); ties to the lower id
        float best = -1.f;
        int best_e = 0x7fffffff;
        for (int e = lane; e < E; e += 32) {
            const float v = prob[e];
            if (v > best) {                                            // ascending e: the first maximum wins
                best = v;
                best_e = e;
            }
        }
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, m);
            const int oe = __shfl_xor_sync(0xffffffffu, best_e, m);
            if (ov > best || (ov == best && oe < best_e)) {
                best = ov;
                best_e = oe;
            }
        }
        if (lane == 0) {
            ids_out[(size_t)t * k + j] = best_e;
            w_out[(size_t)t * k + j] = best * inv;
            prob[best_e] = -2.f;
        }
        __syncwarp();
    }
}

}  // namespace

extern "C" int exmoe_route(const exmoe_shape* shape, const void* hidden_bf16, const void* router_bf16, const float* bias,
                           int T, int32_t* topk_ids, float* topk_weights, void* stream) {
    if (!shape || T < 0) return EXMOE_ERR_ARG;
    if (shape->d_model <= 0 || shape->d_model % 8 || shape->num_experts <= 0 || shape->num_experts > 4096 ||
        shape->top_k <= 0 || shape->top_k > shape->num_experts)
        return EXMOE_ERR_SHAPE;
    if (T == 0) return EXMOE_OK;
    if (!hidden_bf16 || !router_bf16 || !topk_ids || !topk_weights) return EXMOE_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden_bf16) | reinterpret_cast<uintptr_t>(router_bf16)) & 15) return EXMOE_ERR_ARG;
    const size_t smem = (size_t)shape->d_model * 2 + (size_t)shape->num_experts * 4;
    if (smem > 200 * 1024) return EXMOE_ERR_SHAPE;
    static SmemOnce smem_once;
    if (!allow_smem(route_kernel, 200 * 1024, smem_once)) return EXMOE_ERR_CUDA;
    route_kernel<<<T, kRouteThreads, smem, (cudaStream_t)stream>>>(
        (const __nv_bfloat16*)hidden_bf16, (const __nv_bfloat16*)router_bf16, bias, shape->d_model, shape->num_experts,
        shape->top_k, topk_ids, topk_weights);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}

}  // namespace exmoe
