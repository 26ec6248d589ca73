// Shared device-side definitions for the alphakv kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace akv {

constexpr int kMaxD = 256;          // largest head dimension built
constexpr int kMaxHalf = kMaxD / 2;
constexpr int kThreads = 256;       // threads per CTA in the per-event kernels
constexpr int kWarps = kThreads / 32;

// K / V addressing, mirrors akv_layout_t with the page size as a shift.
struct DevLayout {
    int B, L, H, N, d;
    int dtype;
    long long sb, sl, sh, sn;
    int page_size, page_shift;
    const int* table;
    int pps;
    long long s_page, s_page_h, s_page_n;
};

// Slot positions (int32) with broadcastable (b, l, h) strides; p == nullptr: keys already rotated.
struct PosDesc {
    int* p;
    long long sb, sl, sh;
};

// Host-built tables for the score: phi[f] = frac(theta_f / 2 pi) as a 0.64 fixed-point
// fraction of a turn, cw[f] = (1/W) sum_w exp(i w theta_f).
struct ScoreTab {
    unsigned long long phi[kMaxHalf];
    float2 cw[kMaxHalf];
};

__device__ __forceinline__ long long row_offset(const DevLayout& y, int b, int l, int h, int n) {
    if (y.page_size == 0) return b * y.sb + l * y.sl + h * y.sh + n * y.sn;
    const int page = y.table[(long long)b * y.pps + (n >> y.page_shift)];
    return l * y.sl + page * y.s_page + h * y.s_page_h + (long long)(n & (y.page_size - 1)) * y.s_page_n;
}

struct EventId {
    int e, b, l, h;
};
__device__ __forceinline__ EventId decode_event(const DevLayout& y, int e) {
    EventId id;
    id.e = e;
    id.h = e % y.H;
    id.l = (e / y.H) % y.L;
    id.b = e / (y.H * y.L);
    return id;
}

// ---- per-phase cycle stamps (profiling builds only) -------------------------------------------------
// Built with -DAKV_PHASE_CLOCKS (python -m paper_2605_14292_b200.build --phase-clocks, a separate library
// file), thread 0 of every event CTA stores clock64() at the phase boundaries of its kernel into a buffer
// that akv_debug_phase_buffer() registers: kPhaseSlots values per event. The default build compiles the
// stamps to nothing.
constexpr int kPhaseSlots = 16;
#ifdef AKV_PHASE_CLOCKS
__device__ long long* g_phase_buf = nullptr;
__device__ __forceinline__ void phase_stamp(int event, int k) {
    if (threadIdx.x == 0 && g_phase_buf) g_phase_buf[(long long)event * kPhaseSlots + k] = clock64();
}
// cycles spent in a repeated step, summed by thread 0: acc += clock64() at the end, -= at the start
#define AKV_PHASE_ACC_DECL(name) long long name = 0
#define AKV_PHASE_ACC_BEGIN(name) do { if (threadIdx.x == 0) name -= clock64(); } while (0)
#define AKV_PHASE_ACC_END(name) do { if (threadIdx.x == 0) name += clock64(); } while (0)
#define AKV_PHASE_ACC_STORE(event, k, name) do { if (threadIdx.x == 0 && g_phase_buf) g_phase_buf[(long long)(event) * kPhaseSlots + (k)] = name; } while (0)
#else
__device__ __forceinline__ void phase_stamp(int, int) {}
#define AKV_PHASE_ACC_DECL(name)
#define AKV_PHASE_ACC_BEGIN(name)
#define AKV_PHASE_ACC_END(name)
#define AKV_PHASE_ACC_STORE(event, k, name)
#endif

// ---- element access: 4 or 8 consecutive elements widened to fp32 -------------------------------
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&x)[4]) {
    const uint2 w = *reinterpret_cast<const uint2*>(p);
    x[0] = bf16lo(w.x); x[1] = bf16hi(w.x); x[2] = bf16lo(w.y); x[3] = bf16hi(w.y);
}
__device__ __forceinline__ void load4(const float* p, float (&x)[4]) {
    const float4 w = *reinterpret_cast<const float4*>(p);
    x[0] = w.x; x[1] = w.y; x[2] = w.z; x[3] = w.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&x)[8]) {
    const uint4 w = *reinterpret_cast<const uint4*>(p);
    x[0] = bf16lo(w.x); x[1] = bf16hi(w.x); x[2] = bf16lo(w.y); x[3] = bf16hi(w.y);
    x[4] = bf16lo(w.z); x[5] = bf16hi(w.z); x[6] = bf16lo(w.w); x[7] = bf16hi(w.w);
}
__device__ __forceinline__ void load8(const float* p, float (&x)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

// ---- argmax keys: larger value wins, equal values go to the lower index ---------------------------
__device__ __forceinline__ uint32_t orderable(float a) {
    const uint32_t u = __float_as_uint(a);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}
__device__ __forceinline__ unsigned long long pack_key(float a, int j) {
    return ((unsigned long long)orderable(a) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)j);
}
__device__ __forceinline__ int key_index(unsigned long long k) { return (int)(0xFFFFFFFFu - (uint32_t)k); }
__device__ __forceinline__ float key_value(unsigned long long k) { return from_orderable((uint32_t)(k >> 32)); }

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, off);
        v = o > v ? o : v;
    }
    return v;
}

// sum over the G lanes of a lane group (G a power of two <= 32)
__device__ __forceinline__ float group_sum(float v, int G) {
    for (int off = G >> 1; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    return v;
}

__host__ __device__ __forceinline__ int pow2_ceil(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

// 16-byte copies of whole rows, global/shared agnostic
__device__ __forceinline__ void copy16(void* dst, const void* src) {
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
}

}  // namespace akv
