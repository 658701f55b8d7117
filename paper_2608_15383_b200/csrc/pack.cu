// Offline conversion of one expert: Eq. 3 quantiser + packed layout (Section 3.2 of the paper).
//
// One CTA of 256 threads converts one block (16 rows x 128 columns = one scale group per row):
// thread = 16*row + octet reads 8 consecutive BF16 weights (16 bytes), the 16 threads of a row
// reduce the absmax with shuffles, every thread quantises its 8 weights and writes one 32-bit
// word of codes.  HBM-bound: 2 bytes read and 0.516 bytes written per weight.
#include "common.cuh"

#include <mutex>

namespace exmoe {

__global__ void __launch_bounds__(256)
pack_kernel(const __nv_bfloat16* __restrict__ wg, const __nv_bfloat16* __restrict__ wu,
            const __nv_bfloat16* __restrict__ wd, uint8_t* __restrict__ out, int H, int I, int* __restrict__ flag) {
    const int kb13 = H / kGroup, kb2 = I / kGroup;
    const int n13 = (2 * I / kPanelRows) * kb13;           // blocks of the gate/up region
    int b = blockIdx.x;
    const __nv_bfloat16* src;
    int ld, row0, kb;
    if (b < n13) {
        int panel = b / kb13;
        kb = b % kb13;
        src = (panel & 1) ? wu : wg;                        // panels alternate gate, up
        row0 = (panel >> 1) * kPanelRows;
        ld = H;
    } else {
        int bb = b - n13;
        int panel = bb / kb2;
        kb = bb % kb2;
        src = wd;
        row0 = panel * kPanelRows;
        ld = I;
    }
    uint8_t* blk = out + (size_t)b * kBlockBytes;

    const int row = threadIdx.x >> 4, oct = threadIdx.x & 15;
    const uint4 raw = *reinterpret_cast<const uint4*>(src + (size_t)(row0 + row) * ld + kb * kGroup + oct * 8);
    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
    float w[8];
    bool finite = true;
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        w[2 * i] = __uint_as_float(r[i] << 16);
        w[2 * i + 1] = __uint_as_float(r[i] & 0xffff0000u);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        finite = finite && isfinite(w[i]);
        amax = fmaxf(amax, fabsf(w[i]));
    }
#pragma unroll
    for (int m = 8; m >= 1; m >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));   // 16 lanes of a row

    const float s32 = __fdiv_rn(amax, 7.0f);
    const __half s16 = __float2half_rn(s32);
    const float s = __half2float(s16);
    if (!finite || isinf(s)) atomicExch(flag, 1);
    const bool zero = !(s > 0.f);                           // zero group, FP16 underflow (or NaN: flagged)

    uint32_t word = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        float qf = zero ? 0.f : rintf(__fdiv_rn(w[t], s));
        qf = fminf(fmaxf(qf, -8.f), 7.f);
        uint32_t u = (uint32_t)((int)qf + 8) & 0xfu;
        word |= u << (4 * ((t >> 1) + 4 * (t & 1)));
    }
    // word position: half h, lane (q, c), word index 2*set + r  (row = q + 8r, octet = 8h + 4set + c)
    const int h = oct >> 3, set = (oct >> 2) & 1, c = oct & 3, q = row & 7, rr = row >> 3;
    *reinterpret_cast<uint32_t*>(blk + h * 512 + (4 * q + c) * 16 + (2 * set + rr) * 4) = word;
    if (oct == 0) *reinterpret_cast<__half*>(blk + kCodeBytes + (2 * q + rr) * 2) = zero ? __float2half_rn(0.f) : s16;
}

// Non-finite flags of the calls in flight: a ring of words inside the library (exmoe_pack allocates nothing), one word
// per call, so that calls from several host threads on several streams do not share a flag.
constexpr int kPackFlags = 64;
static __device__ int g_pack_flags[kPackFlags];

int* pack_flag_word() {
    static std::mutex mu;
    static int* base[64] = {};
    static unsigned next[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!base[dev]) {
        void* p = nullptr;                                  // the symbol's device address (host code only holds a stand-in)
        if (cudaGetSymbolAddress(&p, g_pack_flags) != cudaSuccess || !p) {
            cudaGetLastError();
            return nullptr;
        }
        base[dev] = static_cast<int*>(p);
    }
    return base[dev] + (next[dev]++ % kPackFlags);
}

int launch_pack(const exmoe_shape& s, const void* wg, const void* wu, const void* wd, void* out, int* d_flag,
                cudaStream_t st) {
    const int H = s.d_model, I = s.d_ff;
    const int nblocks = (2 * I / kPanelRows) * (H / kGroup) + (H / kPanelRows) * (I / kGroup);
    pack_kernel<<<nblocks, 256, 0, st>>>((const __nv_bfloat16*)wg, (const __nv_bfloat16*)wu,
                                         (const __nv_bfloat16*)wd, (uint8_t*)out, H, I, d_flag);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? EXMOE_OK : EXMOE_ERR_CUDA;
}

}  // namespace exmoe
