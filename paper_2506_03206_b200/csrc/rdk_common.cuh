// Shared device/host helpers of the RDK library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rdk.h"

namespace rdk {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kVec = 8;                 // consecutive tokens one thread handles per step
constexpr int kRowThreads = 512;        // threads of a row CTA
constexpr int kRowWarps = kRowThreads / 32;
constexpr int kTile = kRowThreads * kVec;   // tokens one CTA covers per step (4096)
constexpr int kSeg = 32 * kVec;             // tokens one warp covers per step (256): one CDF segment

// ---- kept-id index layout (device buffer built by rdk_prepare_ids) ---------------------------
// [0, 256)           header: int32 magic, N, n, n_valid, dup, identity, plan, ...
// [256, ..)          uint32 mask[words]    bit t set <=> token t is a kept id inside [0, N)
// then               int32  rank[words]    number of set bits in all earlier words
// then               int32  slot[n]        slot[r] = drafter index of the r-th smallest valid id
// then               int32  ids[n]         copy of the caller's kept ids
// then, for the target element sizes 2 and 4 bytes (v = 0, 1), the tables of the streaming kernels:
//                    int4   segdesc[v][256]   per segment: first kept slot r0 (even), kept slots, table start, dummy
//                    uint16 goff[v][..]       per kept slot: byte offset of its target logit in the CTA's slice
constexpr int kIdxMagic = 0x52444B32;   // "RDK2"
enum { kHdrMagic = 0, kHdrN = 1, kHdrn = 2, kHdrValid = 3, kHdrDup = 4, kHdrIdentity = 5, kHdrPlan = 6 };

// ---- segmentation of the vocabulary by the streaming kernels ---------------------------------
// A row is shared by C CTAs of kStreamWarps warps; warp w of CTA c owns the Lw consecutive tokens
// ("segment") starting at (c * kStreamWarps + w) * Lw.  Lw is a whole number nv of 16-byte vectors
// per lane.  Depends on N and the target element size only, so the per-segment tables can be built
// when the kept ids are prepared.
#ifndef RDK_STREAM_WARPS
#define RDK_STREAM_WARPS 16
#endif
constexpr int kStreamWarps = RDK_STREAM_WARPS;
constexpr int kStreamMaxGroup = 16;                              // CTAs that share a row
constexpr int kStreamMaxSeg = kStreamMaxGroup * kStreamWarps;    // 256
constexpr int kStreamMinN = 4096;
struct StreamSegs { int C, Lw, nv; };
inline bool stream_segments(int N, size_t es, StreamSegs& g) {
    if (N < kStreamMinN) return false;
    const int vt = 32 * (int)(16 / es);    // tokens one warp covers with one 16-byte vector per lane
    int C = (N + 64 * vt - 1) / (64 * vt);     // slices of about 64 vectors per lane (32 KB of logits)
    if (C > kStreamMaxGroup) C = kStreamMaxGroup;
    g.nv = (N + C * kStreamWarps * vt - 1) / (C * kStreamWarps * vt);
    g.Lw = g.nv * vt;
    g.C = (N + kStreamWarps * g.Lw - 1) / (kStreamWarps * g.Lw);          // no CTA of a group without tokens
    // offsets into a CTA's slice (and the spare slot behind it) are 16-bit
    return (size_t)kStreamWarps * g.Lw * es + 16 <= 65535;
}

struct KeptIndexView {
    const int32_t* header;
    const uint32_t* mask;
    const int32_t* rank;
    const int32_t* slot;
    const int32_t* ids;
    const int4* segdesc[2];
    const uint16_t* goff[2];
    int words;
};

__host__ __device__ inline int idx_words(int N) { return ((N + 31) / 32 + 63) & ~63; }  // padded
__host__ __device__ inline size_t idx_align(size_t x) { return (x + 255) & ~size_t(255); }
__host__ __device__ inline size_t idx_off_mask() { return 256; }
__host__ __device__ inline size_t idx_off_rank(int N) { return idx_off_mask() + idx_align(size_t(idx_words(N)) * 4); }
__host__ __device__ inline size_t idx_off_slot(int N) { return idx_off_rank(N) + idx_align(size_t(idx_words(N)) * 4); }
__host__ __device__ inline size_t idx_off_ids(int N, int n) { return idx_off_slot(N) + idx_align(size_t(n) * 4); }
// every segment's run of kept slots is padded to a multiple of 64 (and may start one slot early)
__host__ __device__ inline size_t idx_goff_slots(int n) { return size_t(n) + size_t(kStreamMaxSeg) * 66; }
__host__ __device__ inline size_t idx_plan_bytes(int n) { return idx_align(size_t(kStreamMaxSeg) * 16) + idx_align(idx_goff_slots(n) * 2); }
__host__ __device__ inline size_t idx_off_plan(int N, int n, int v) { return idx_off_ids(N, n) + idx_align(size_t(n) * 4) + size_t(v) * idx_plan_bytes(n); }
__host__ __device__ inline size_t idx_bytes(int N, int n) { return idx_off_plan(N, n, 2); }

inline KeptIndexView make_view(const void* base, int N, int n) {
    const char* b = static_cast<const char*>(base);
    KeptIndexView v;
    v.header = reinterpret_cast<const int32_t*>(b);
    v.mask = reinterpret_cast<const uint32_t*>(b + idx_off_mask());
    v.rank = reinterpret_cast<const int32_t*>(b + idx_off_rank(N));
    v.slot = reinterpret_cast<const int32_t*>(b + idx_off_slot(N));
    v.ids = reinterpret_cast<const int32_t*>(b + idx_off_ids(N, n));
    for (int k = 0; k < 2; ++k) {
        v.segdesc[k] = reinterpret_cast<const int4*>(b + idx_off_plan(N, n, k));
        v.goff[k] = reinterpret_cast<const uint16_t*>(b + idx_off_plan(N, n, k) + idx_align(size_t(kStreamMaxSeg) * 16));
    }
    v.words = idx_words(N);
    return v;
}

// What rdk_prepare_ids learnt about the index it built at `kept_index` for (N, n): 1 when the kept ids
// are ascending and all inside [0, N) (rank = drafter index), 0 when not, -1 when this process never
// built an index for that (N, n) at that address.  Kernels that rely on it re-check the header on the device.
void note_index_order(const void* kept_index, int N, int n, bool ascending_valid);
int index_order(const void* kept_index, int N, int n);

// ---- host-side error plumbing ------------------------------------------------------------------
void set_error(const char* fmt, ...);
int cuda_fail(cudaError_t e, const char* what);
int check_arch();                        // RDK_OK or RDK_ERR_ARCH / RDK_ERR_CUDA

#define RDK_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) return ::rdk::cuda_fail(e__, #call); \
    } while (0)

// ---- device helpers ---------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Load kVec consecutive elements row[base .. base+8) as floats.  `vec_ok` says that the row base
// is 16-byte aligned; elements at or beyond `len` read as `fill`.
template <typename T>
__device__ __forceinline__ void load8(const T* __restrict__ row, int base, int len, bool vec_ok,
                                      float fill, float (&v)[kVec]);

template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* __restrict__ row, int base,
                                                     int len, bool vec_ok, float fill,
                                                     float (&v)[kVec]) {
    if (vec_ok && base + kVec <= len) {
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(row + base));
        v[0] = bf16_lo(q.x); v[1] = bf16_hi(q.x); v[2] = bf16_lo(q.y); v[3] = bf16_hi(q.y);
        v[4] = bf16_lo(q.z); v[5] = bf16_hi(q.z); v[6] = bf16_lo(q.w); v[7] = bf16_hi(q.w);
    } else {
#pragma unroll
        for (int k = 0; k < kVec; ++k) v[k] = (base + k < len) ? __bfloat162float(row[base + k]) : fill;
    }
}

template <>
__device__ __forceinline__ void load8<float>(const float* __restrict__ row, int base, int len,
                                             bool vec_ok, float fill, float (&v)[kVec]) {
    if (vec_ok && base + kVec <= len) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(row + base));
        const float4 b = __ldg(reinterpret_cast<const float4*>(row + base + 4));
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
        for (int k = 0; k < kVec; ++k) v[k] = (base + k < len) ? row[base + k] : fill;
    }
}
#endif  // __CUDACC__

}  // namespace rdk
