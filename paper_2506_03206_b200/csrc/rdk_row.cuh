// Declarations shared by the row kernels (generic one-CTA-per-row kernel and the streaming kernels).
#pragma once

#include <math.h>

#include "rdk_common.cuh"

namespace rdk {

struct RowParams {
    int N, n, rows, trials;
    const void* target;  long long target_stride;
    const void* drafter; long long drafter_stride;
    const float* w;      long long w_stride;
    const float* uniforms;
    const void* prior; long long prior_stride;   // logits that replace the target inside Eq. rdk-taylor (NULL: none)
    const int32_t* header; const uint32_t* mask; const int32_t* rank; const int32_t* slot; const int32_t* ids;
    int32_t* draft_token; int32_t* out_token; uint8_t* accepted; float* accept_prob;
    float* alpha; float* theta; float* S; float* residual_mass; float* qtilde;
    int32_t* status_word;
    int num_tiles;
    int w_as_given;        // precomputed-w mode: q~ = w itself (no division by its sum)
    // streaming path only
    int positions;
    int32_t* accepted_len;
    float* rec;            // per-row records in the workspace
    int32_t* counters;     // per (sequence, trial) arrival counters in the workspace
    unsigned char* xrec;   // per (row, CTA of the group) published partial records and flags in the workspace
};


// running (max, sum) pair of a soft-max denominator; `b` is a second sum on the same scale
struct MS { float m, s, b; };

__device__ __forceinline__ MS ms_combine(const MS& x, const MS& y) {
    MS r;
    r.m = fmaxf(x.m, y.m);
    if (r.m == -INFINITY) { r.s = 0.f; r.b = 0.f; return r; }
    const float fx = ex2((x.m - r.m) * kLog2e), fy = ex2((y.m - r.m) * kLog2e);
    r.s = x.s * fx + y.s * fy;
    r.b = x.b * fx + y.b * fy;
    return r;
}
__device__ __forceinline__ void ms_push(MS& a, float x) {
    if (x > a.m) { a.s = a.s * ex2((a.m - x) * kLog2e) + 1.f; a.m = x; }
    else if (x > -INFINITY) a.s += ex2((x - a.m) * kLog2e);
}
__device__ __forceinline__ MS ms_warp(MS v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MS t;
        t.m = __shfl_xor_sync(0xffffffffu, v.m, o);
        t.s = __shfl_xor_sync(0xffffffffu, v.s, o);
        t.b = __shfl_xor_sync(0xffffffffu, v.b, o);
        v = ms_combine(v, t);
    }
    return v;
}

// Inclusive fp64 prefix sums of seg[0..count) into cdf[], done by one warp; returns the total.
__device__ __forceinline__ double warp_scan_segments(const float* seg, double* cdf, int count, int lane) {
    const int per = (count + 31) / 32;
    const int lo = lane * per, hi = min(count, lo + per);
    double loc = 0.0;
    for (int s = lo; s < hi; ++s) loc += (double)seg[s];
    double incl = loc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    double run = incl - loc;
    for (int s = lo; s < hi; ++s) { run += (double)seg[s]; cdf[s] = run; }
    return __shfl_sync(0xffffffffu, incl, 31);
}

// first s with cdf[s] > thr (cdf non-decreasing); count if none
__device__ __forceinline__ int first_above(const double* cdf, int count, double thr) {
    int lo = 0, hi = count;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (cdf[mid] > thr) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// Within one 256-token segment held as x[kVec] per lane: the first token whose inclusive prefix
// sum exceeds rem and whose weight is positive; if rounding leaves none, the last positive token.
// Returns lane * kVec + k (same value in all lanes), or -1 when the segment has no positive weight.
__device__ __forceinline__ int pick_in_segment(const float (&x)[kVec], float rem, int lane) {
    float c[kVec];
    float run = 0.f;
#pragma unroll
    for (int k = 0; k < kVec; ++k) { run += x[k]; c[k] = run; }
    float incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    const float pre = incl - run;
    int hit = -1, last_pos = -1;
#pragma unroll
    for (int k = kVec - 1; k >= 0; --k) {
        if (x[k] > 0.f) {
            if (last_pos < 0) last_pos = k;
            if (pre + c[k] > rem) hit = k;
        }
    }
    const uint32_t hits = __ballot_sync(0xffffffffu, hit >= 0);
    if (hits) {
        const int src = __ffs(hits) - 1;
        return src * kVec + __shfl_sync(0xffffffffu, hit, src);
    }
    const uint32_t pos = __ballot_sync(0xffffffffu, last_pos >= 0);
    if (!pos) return -1;
    const int src = 31 - __clz(pos);
    return src * kVec + __shfl_sync(0xffffffffu, last_pos, src);
}


// Launches the streaming kernel for the linear path when the problem qualifies; returns
// cudaErrorNotSupported (and launches nothing) when the one-CTA-per-row kernel has to be used.
cudaError_t launch_stream_linear(RowParams P, int tz, int ty, int kind, int batch, void* ws, size_t ws_bytes, cudaStream_t s);
size_t stream_workspace_bytes(int rows, int batch, int trials);
// Why a problem cannot take the streaming kernel (a static string), or NULL when it can.  Host only.
const char* stream_ineligible(const RowParams& P, int tz, int ty, int kind, int batch, const void* ws, size_t ws_bytes);
// Failed tries after which a device-side wait of the streaming kernel gives up (0: the default).
void set_stream_spin_limit(unsigned limit);

}  // namespace rdk
