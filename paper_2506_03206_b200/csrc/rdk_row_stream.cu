// Streaming form of the linear-time path (Eq. rdk-taylor + Algorithm 4 steps 4-8) for N >= 4096
// and kept ids in ascending order: one persistent kernel, one launch per call.
//
// The grid is G groups of C CTAs, one CTA per SM.  Group g takes rows g, g + G, ...; within a row,
// streaming warp w of CTA c owns the contiguous token range ("segment") s = 16 c + w.  A CTA has 20
// warps and no block-wide barrier in its row loop:
//   load warp      : per row, one bulk copy (TMA) of the CTA's slice of the target logits and one per
//                    streaming warp of the matching contiguous run of drafter values, into a ring of
//                    NS shared-memory stages, so a row is read from HBM exactly once.
//   16 streaming warps, first visit A(row): maximum and sum of e = exp(z - max) over the segment, and
//                    over the segment's kept tokens sum e_z, sum e_y, sum e_z e_y; the (e_z, e_y)
//                    pairs are cached.  Second visit B(row), NB - 1 rows later: sum min(p, q~) over
//                    the cached pairs, when the row's scalars are known.
//   publish warp   : folds the CTA's 16 warp records of a row into one and publishes it in global
//                    memory as five 64-bit words, each a value paired with a per-call tag (so every
//                    word validates itself and no fence is needed); NB rows later, writes the row's
//                    per-segment sums and raises the CTA's flag for that row.
//   collect warp   : polls the C records of a row and leaves the row scalars and every warp's scale
//                    factors in shared memory for the second visits.
//   draw warp      : CTA c of a group turns rows c, c + C, ... of the group into draws once all C
//                    flags of the row are up: prefix sums over the segments, locate the segment of the
//                    draft draw, re-read that one segment (still in L2), pick the token, run the
//                    rejection test, on rejection the same for the residual draw, write the outputs
//                    and count the accepted prefix of the sequence.
// The exchange of a row costs about two first visits of latency; with the second visit trailing by
// NB - 1 rows and the exchange and the draws in warps of their own, both are off the streaming
// warps' critical path.  Everything that depends only on (N, n, kept ids, element size) -- which
// kept slots belong to which segment and where their target logits sit in the CTA's slice -- is
// tabulated once by rdk_prepare_ids and read from the kept-id index.
//
// Arithmetic, with p = softmax(z), q' = TLI(softmax(y)), x_j = p_j / N <= 2^-12:
//   w_j = (N q'_j + theta p_j) / (N + p_j) = (q'_j + theta x_j) / (1 + x_j)
//       = q'_j + x_j (theta - q'_j) + O(x_j^2)          (dropped terms are below 2^-24 of the total)
// * A token the drafter does not keep has q'_j = 0, hence w_j / S < p_j: its share of
//   alpha = sum min(p, q~) is w_j / S and its residual is p_j - w_j / S.  Such tokens enter only
//   through sum p_j per segment, which comes out of the soft-max sweep itself.
// * S = sum_j w_j = 1 + O(N^-2), because sum q' = 1 and sum q'_j p_j = theta cancel the
//   first-order terms; it is taken as 1.
#include <atomic>
#include <chrono>

#include "rdk_row.cuh"

namespace rdk {

constexpr int kSW = kStreamWarps;        // streaming warps (= segments) per CTA
constexpr int kWPublish = kSW, kWCollect = kSW + 1, kWLoad = kSW + 2;
constexpr int kSThreads = (kSW + 3) * 32;
constexpr int kMaxGroup = kStreamMaxGroup;   // CTAs that share a row
constexpr int kMaxSeg = kStreamMaxSeg;       // 256
constexpr unsigned kSpinLimitDefault = 1u << 17;   // with up to 2 us per try: a quarter of a second
constexpr int kMaxChunks = 128;          // 256-token chunks per segment
constexpr int kMaxNB = 8;                // most rows whose records and caches are alive at once (StreamGeo::NB)
constexpr int kTmemCols = 512;           // tensor memory columns of an SM (128 lanes x 512 columns x 32 bits)
constexpr int kTmemWarpCols = kTmemCols / (kSW / 4);   // columns of a streaming warp: four warps share a 32-lane quarter
constexpr int kXrecBytes = 64;           // one published CTA record: five (value, tag) words, padded
constexpr int kRecFloats = 16 + 4 * kMaxSeg;   // one row's record: 16 scalars, then per segment the sums of w, min(p, q~),
                                         // max(0, p - q~) and p
constexpr int kFastNit = 64 / kSW;       // 16-byte vectors per lane in a segment of the common length
constexpr int kMaxFastSteps = 6;         // kept-token passes of up to this many steps are unrolled, their offsets in registers

// scalars of a row's record
enum { kRecOffg = 0, kRecInvZp, kRecYoffg, kRecInvZq, kRecTheta };

struct Scal { float offg, inv_zp, yoffg, inv_zq, theta, inv_n, inv_s; };

struct StreamGeo {
    int C, G;              // CTAs per group, groups
    int Lw;                // tokens per segment: nv vectors of 16 bytes per lane
    int nv;
    int NS;                // stages
    int NB;                // rows whose records and caches are alive at once: the second visit of a row
                           // follows its first visit NB - 1 rows later
    int ycap;              // kept-token slots per warp that are staged and cached (multiple of 64)
    int ystage;            // bytes of a warp's drafter region in a stage
    uint32_t tag;          // value that marks a word in the workspace as written by this call
    unsigned spin_limit;   // failed tries after which a wait gives up
    const int4* segdesc;   // per segment: first slot r0, slots in use, start in goff[], dummy
    const uint16_t* goff;  // per slot: byte offset of its target logit in the CTA's slice
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <typename T> __device__ __forceinline__ T neg_inf();
template <> __device__ __forceinline__ float neg_inf<float>() { return -INFINITY; }
template <> __device__ __forceinline__ __nv_bfloat16 neg_inf<__nv_bfloat16>() { return __float2bfloat16_rn(-INFINITY); }
template <typename T> __device__ __forceinline__ T zero_of();
template <> __device__ __forceinline__ float zero_of<float>() { return 0.f; }
template <> __device__ __forceinline__ __nv_bfloat16 zero_of<__nv_bfloat16>() { return __float2bfloat16_rn(0.f); }

// w_j for given p_j and q'_j:  (q' + theta x) (1 - x + x^2),  x = p / N
__device__ __forceinline__ float taylor_w(const Scal& c, float p, float qp) {
    const float x = p * c.inv_n;
    return fmaf(c.theta, x, qp) * fmaf(x, x - 1.f, 1.f);
}

// ---- packed fp32 pairs ---------------------------------------------------------------------------
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(*reinterpret_cast<unsigned long long*>(&d))
        : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)),
          "l"(*reinterpret_cast<unsigned long long*>(&c)));
    return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    float2 d;
    asm("add.rn.f32x2 %0, %1, %2;"
        : "=l"(*reinterpret_cast<unsigned long long*>(&d))
        : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)));
    return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
    float2 d;
    asm("mul.rn.f32x2 %0, %1, %2;"
        : "=l"(*reinterpret_cast<unsigned long long*>(&d))
        : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)));
    return d;
}
__device__ __forceinline__ float2 splat(float v) { return make_float2(v, v); }
__device__ __forceinline__ float2 ex2_2(float2 x) { return make_float2(ex2(x.x), ex2(x.y)); }

// ---- shared-memory access by 32-bit shared address -----------------------------------------------
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t a, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

// ---- tensor memory as a per-warp scratch-pad -------------------------------------------------------
// Lane i of a warp reads and writes 32-bit words of TMEM lane 32 (warp % 4) + i; four consecutive columns
// per access.  Nothing here involves the tensor cores: the 256 KB that would hold MMA accumulators hold
// the cached (e_z, e_y) pairs of the rows in flight instead, which leaves shared memory to the stages.
__device__ __forceinline__ void tmem_st4(uint32_t taddr, float a, float b, float c, float d) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(taddr), "r"(__float_as_uint(a)), "r"(__float_as_uint(b)), "r"(__float_as_uint(c)), "r"(__float_as_uint(d)) : "memory");
}
__device__ __forceinline__ uint4 tmem_ld4(uint32_t taddr) {
    uint4 v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(taddr) : "memory");
    return v;
}

// one target logit at shared byte address a, as fp32
template <typename TZ> __device__ __forceinline__ float lds_z(uint32_t a);
template <> __device__ __forceinline__ float lds_z<__nv_bfloat16>(uint32_t a) { return __uint_as_float(lds16(a) << 16); }
template <> __device__ __forceinline__ float lds_z<float>(uint32_t a) { return __uint_as_float(lds32(a)); }

// two consecutive drafter values at shared byte address a (aligned to the pair), as fp32
template <typename TY> __device__ __forceinline__ float2 lds_ypair(uint32_t a);
template <> __device__ __forceinline__ float2 lds_ypair<__nv_bfloat16>(uint32_t a) {
    const uint32_t w = lds32(a);
    return make_float2(bf16_lo(w), bf16_hi(w));
}
template <> __device__ __forceinline__ float2 lds_ypair<float>(uint32_t a) {
    const uint2 w = lds64(a);
    return make_float2(__uint_as_float(w.x), __uint_as_float(w.y));
}

// maximum of the 8 logits (bf16) / 4 logits (fp32) in one 16-byte vector
template <typename TZ> struct MaxAcc;
template <> struct MaxAcc<float> {
    float m = -INFINITY;
    __device__ __forceinline__ void push(uint4 q) {
        m = fmaxf(fmaxf(m, __uint_as_float(q.x)), fmaxf(__uint_as_float(q.y), fmaxf(__uint_as_float(q.z), __uint_as_float(q.w))));
    }
    __device__ __forceinline__ float result() const { return m; }
};
template <> struct MaxAcc<__nv_bfloat16> {
    __nv_bfloat162 ma = __float2bfloat162_rn(-INFINITY), mb = __float2bfloat162_rn(-INFINITY);
    __device__ __forceinline__ void push(uint4 q) {
        ma = __hmax2(ma, *reinterpret_cast<const __nv_bfloat162*>(&q.x));
        mb = __hmax2(mb, *reinterpret_cast<const __nv_bfloat162*>(&q.y));
        ma = __hmax2(ma, *reinterpret_cast<const __nv_bfloat162*>(&q.z));
        mb = __hmax2(mb, *reinterpret_cast<const __nv_bfloat162*>(&q.w));
    }
    __device__ __forceinline__ float result() const {
        const __nv_bfloat162 m2 = __hmax2(ma, mb);
        return fmaxf(__low2float(m2), __high2float(m2));
    }
};

// sum of e = 2^(z log2e + off) over the logits of one 16-byte vector, two packed accumulators.  (Evaluating a
// share of the exponentials by a polynomial on the FMA pipe relieves the special-function unit but costs issue
// slots, which are the scarcer resource in this kernel: measured, it does not pay.)
template <typename TZ> __device__ __forceinline__ void exp_sum_vec(uint4 q, float2 scale, float2 off, float2& Ea, float2& Eb);
template <> __device__ __forceinline__ void exp_sum_vec<__nv_bfloat16>(uint4 q, float2 scale, float2 off, float2& Ea, float2& Eb) {
    const float2 e0 = ex2_2(ffma2(make_float2(bf16_lo(q.x), bf16_hi(q.x)), scale, off));
    const float2 e1 = ex2_2(ffma2(make_float2(bf16_lo(q.y), bf16_hi(q.y)), scale, off));
    const float2 e2 = ex2_2(ffma2(make_float2(bf16_lo(q.z), bf16_hi(q.z)), scale, off));
    const float2 e3 = ex2_2(ffma2(make_float2(bf16_lo(q.w), bf16_hi(q.w)), scale, off));
    Ea = fadd2(Ea, e0); Eb = fadd2(Eb, e1); Ea = fadd2(Ea, e2); Eb = fadd2(Eb, e3);
}
template <> __device__ __forceinline__ void exp_sum_vec<float>(uint4 q, float2 scale, float2 off, float2& Ea, float2& Eb) {
    const float2 e0 = ex2_2(ffma2(make_float2(__uint_as_float(q.x), __uint_as_float(q.y)), scale, off));
    const float2 e1 = ex2_2(ffma2(make_float2(__uint_as_float(q.z), __uint_as_float(q.w)), scale, off));
    Ea = fadd2(Ea, e0); Eb = fadd2(Eb, e1);
}

// Wait for the phase of `bar` with the given parity.  Each try may park the warp in hardware for up to
// HINT_NS nanoseconds (it wakes as soon as the phase completes), so a waiting warp issues next to nothing;
// after `limit` failed tries the wait gives up and the host reads RDK_ERR_TIMEOUT.
template <int HINT_NS = 2000>
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, int* fail, unsigned limit) {
    unsigned spins = 0;
    uint32_t done = 0;
    while (!done) {
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(bar), "r"(parity), "r"((uint32_t)HINT_NS) : "memory");
        if (!done && (++spins > limit || *reinterpret_cast<volatile int*>(fail))) {
            atomicExch(fail, 1);
            break;
        }
    }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// (value, tag) words in global memory: one 64-bit relaxed access each, so a reader sees a value
// together with the tag that was stored with it
__device__ __forceinline__ void st_tagged(unsigned char* p, float v, uint32_t tag) {
    const unsigned long long w = ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v);
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(w) : "memory");
}
__device__ __forceinline__ unsigned long long ld_tagged(const unsigned char* p) {
    unsigned long long w;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(w) : "l"(p) : "memory");
    return w;
}
__device__ __forceinline__ int ld_volatile_s32(const int* p) {
    int v;
    asm volatile("ld.volatile.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}

// Sums of four per-lane values over the warp with 6 shuffles: afterwards lanes 0-7 hold the total of
// v0, lanes 8-15 of v1, lanes 16-23 of v2, lanes 24-31 of v3.
__device__ __forceinline__ float warp_sum4(float v0, float v1, float v2, float v3, int lane) {
    const bool up = lane & 16;
    float a = up ? v2 : v0, b = up ? v3 : v1;
    a += __shfl_xor_sync(0xffffffffu, up ? v0 : v2, 16);
    b += __shfl_xor_sync(0xffffffffu, up ? v1 : v3, 16);
    const bool odd = lane & 8;
    float k = odd ? b : a;
    k += __shfl_xor_sync(0xffffffffu, odd ? a : b, 8);
    k += __shfl_xor_sync(0xffffffffu, k, 4);
    k += __shfl_xor_sync(0xffffffffu, k, 2);
    k += __shfl_xor_sync(0xffffffffu, k, 1);
    return k;
}
__device__ __forceinline__ float warp_max_redux(float v) {
    float m;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(v));
    return m;
}

// Combine per-lane partial soft-max records (sum e, sum e_y, sum e e_y on the scales m, my) over
// the warp; lanes without a record pass m = my = -inf and zeros.
__device__ __forceinline__ void combine_records(float& E1, float& Zq, float& th, float& m, float& my, int lane) {
    const float mm = warp_max_redux(m), mmy = warp_max_redux(my);
    const float f = m > -INFINITY ? ex2((m - mm) * kLog2e) : 0.f;
    const float g = my > -INFINITY ? ex2((my - mmy) * kLog2e) : 0.f;
    const float tot = warp_sum4(E1 * f, Zq * g, th * f * g, 0.f, lane);
    E1 = __shfl_sync(0xffffffffu, tot, 0); Zq = __shfl_sync(0xffffffffu, tot, 8); th = __shfl_sync(0xffffffffu, tot, 16);
    m = mm; my = mmy;
}

// ------------------------------------------------------------------------------------------------
// helpers of the draw kernel (Algorithm 4 steps 4-8)
// ------------------------------------------------------------------------------------------------
struct DrawCtx {
    const void* zrow; const void* yrow; bool zvec;
    const uint32_t* mask; const int32_t* rank;
    int N;
    Scal c;
};

// p and w of the 8 tokens starting at global token jb (a multiple of 8).  The drafter values of the kept
// tokens among them are fetched by eight independent loads (tokens that are not kept re-read the first
// fetched index), so that one round trip serves them all.
template <typename TZ, typename TY, int KIND>
__device__ __forceinline__ void draw_pw(const DrawCtx& d, int jb, float (&p)[kVec], float (&w)[kVec]) {
    float z[kVec];
    load8<TZ>(static_cast<const TZ*>(d.zrow), jb, d.N, d.zvec, -INFINITY, z);
    const uint32_t word = __ldg(d.mask + (jb >> 5));
    const int rbase = __ldg(d.rank + (jb >> 5));          // issued together with the mask and the logits
    const int sh = jb & 31;
    const uint32_t mb = (word >> sh) & 0xffu;
    const int r0 = rbase + __popc(word & ((1u << sh) - 1u));
    const int rfirst = mb ? r0 : 0;
    float y[kVec];
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        const bool kept = (mb >> k) & 1u;
        const int r = kept ? r0 + __popc(mb & ((1u << k) - 1u)) : rfirst;    // ascending kept ids: rank = drafter index
        y[k] = to_float<TY>(static_cast<const TY*>(d.yrow)[r]);
    }
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        p[k] = ex2(fmaf(z[k], kLog2e, d.c.offg)) * d.c.inv_zp;
        const bool kept = (mb >> k) & 1u;
        const float qp = kept ? (KIND == RDK_LOGITS ? ex2(fmaf(y[k], kLog2e, d.c.yoffg)) : y[k]) * d.c.inv_zq : 0.f;
        w[k] = taylor_w(d.c, p[k], qp);
    }
}

enum { kPickW = 0, kPickR = 1, kPickP = 2 };

template <typename TZ, typename TY, int KIND>
__device__ __forceinline__ void draw_x(const DrawCtx& d, int what, int jb, int seg_end, float (&p)[kVec], float (&w)[kVec], float (&x)[kVec]) {
#pragma unroll
    for (int k = 0; k < kVec; ++k) { p[k] = 0.f; w[k] = 0.f; x[k] = 0.f; }
    if (jb >= seg_end) return;
    draw_pw<TZ, TY, KIND>(d, jb, p, w);
#pragma unroll
    for (int k = 0; k < kVec; ++k)
        x[k] = what == kPickW ? w[k] : (what == kPickR ? fmaxf(0.f, p[k] - w[k] * d.c.inv_s) : p[k]);
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
// NIT > 0: a segment is exactly NIT 16-byte vectors per lane, kept in registers between the maximum
// and the exponential pass; NIT = 0: any segment length, two passes over shared memory.
// NST > 0: the kept-token passes take exactly NST steps of 64 slots, unrolled, with the slots' offsets in
// registers; NST = 0: any number of steps, offsets in shared memory.
template <typename TZ, typename TY, int KIND, int NIT, int NST>
__global__ void __launch_bounds__(kSThreads, 1)
rdk_stream_kernel(const RowParams P, const StreamGeo g) {
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ __align__(16) float wrec[kMaxNB][kSW][8];   // [row mod NB][warp]: sum e, sum e_z, sum e_y, sum e_z e_y (kept), scale of z, scale of y
    __shared__ __align__(16) float scal[kMaxNB][8];        // [row mod NB]: theta
    __shared__ __align__(8) float2 fzy[kMaxNB][kSW];       // [row mod NB][warp]: factors that turn the warp's cached e_z, e_y into p, q'
    __shared__ float akv[kMaxNB][kSW];                     // [row mod NB][warp]: sum of min(p, q~) over the warp's kept tokens
    __shared__ __align__(8) unsigned long long abar[kMaxNB];   // [row mod NB]: the 16 warp records of the row are in wrec[]
    __shared__ __align__(8) unsigned long long rbar[kMaxNB];   // [row mod NB]: scal[] and fzy[] of the row are set
    __shared__ __align__(8) unsigned long long bbar[kMaxNB];   // [row mod NB]: akv[] of the row is set
    __shared__ __align__(8) unsigned long long pbar[16];    // [row mod 16]: the publish warp has parked the row in pend[]
    __shared__ __align__(16) float pend[16][kSW][8];    // publish and collect warps only, [row mod 16][warp]: the warp's sums, its factors, theta, a row scalar
    __shared__ int fail;
    __shared__ uint32_t tmem_base_s;                       // base address of the CTA's tensor memory (unrolled route)
    constexpr bool kTmem = NST > 0;                        // the pair cache lives in tensor memory, not in shared memory

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);     // the same in every lane, and the compiler knows it
    const int grp = blockIdx.x / g.C, crank = blockIdx.x % g.C;

    // header of the index and this warp's segment descriptor, all requested before any of them is looked at
    const int4 hdr = __ldg(reinterpret_cast<const int4*>(P.header));            // magic, N, n, valid ids
    const int4 hdr2 = __ldg(reinterpret_cast<const int4*>(P.header) + 1);       // dup, identity, plan
    // streaming warp w: its own segment; service warps: lane w looks after warp w's segment
    const int seg = crank * kSW + (warp < kSW ? warp : (lane & (kSW - 1)));
    const int4 sd = __ldg(g.segdesc + seg);                                     // r0, kcp, start in goff[], dummy
    if (hdr.x != kIdxMagic || hdr.y != P.N || hdr.z != P.n || !hdr2.y || hdr.w != P.n ||
        !(hdr2.z & (sizeof(TZ) == 2 ? 1 : 2))) {
        // not the index the host was told about: the same decision in every CTA; nothing is in flight yet
        if (tid == 0 && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_INVALID_ARG);
        return;
    }
    // the next kernel of the stream may be scheduled as soon as this one leaves room; it waits for this
    // whole grid before it touches its inputs or the workspace
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    constexpr int kZPer = 16 / (int)sizeof(TZ);          // logits per 16 bytes
    const int rows_g = grp < P.rows ? (P.rows - grp + g.G - 1) / g.G : 0;
    const float inv_n = 1.f / (float)P.N;
    const unsigned spin_limit = g.spin_limit;

    // shared memory: NS stages of [the CTA's slice of a target row | 16 bytes of -inf | one drafter
    // region per warp], then per warp the (e_z, e_y) cache (NB rows) and (NST = 0) the gather offsets, then barriers
    const uint32_t zslice = (uint32_t)kSW * (uint32_t)g.Lw * (uint32_t)sizeof(TZ);
    const uint32_t stage = zslice + 16u + (uint32_t)kSW * (uint32_t)g.ystage;
    const uint32_t off_cache = (uint32_t)g.NS * stage;
    const int nb = g.NB, defer = g.NB - 1;
    const uint32_t off_goff = off_cache + (kTmem ? 0u : (uint32_t)kSW * (uint32_t)nb * (uint32_t)g.ycap * 8u);
    const uint32_t off_bar = off_goff + (NST > 0 ? 0u : (uint32_t)kSW * (uint32_t)g.ycap * 2u);
    const uint32_t dsm_a = smem_u32(dsm);
    const uint32_t full_a = dsm_a + off_bar, empty_a = full_a + 8u * (uint32_t)g.NS;
    const int nst = NST > 0 ? NST : g.ycap >> 6;           // steps of 32 lanes x 2 slots in a kept-token pass

    if (tid == 0) {
        fail = 0;
        for (int k = 0; k < kMaxNB; ++k) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&abar[k])), "r"(kSW));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&rbar[k])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&bbar[k])), "r"(kSW));
        }
        for (int k = 0; k < 16; ++k) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&pbar[k])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // per-warp quantities of the streaming warps (taken from lane 0 so that the compiler knows they are uniform)
    const int w_r0 = __shfl_sync(0xffffffffu, sd.x, 0), w_kcp = __shfl_sync(0xffffffffu, sd.y, 0);
    const int w_gstart = __shfl_sync(0xffffffffu, sd.z, 0), w_dummy = __shfl_sync(0xffffffffu, sd.w, 0);
    const int w_kcs = min(w_kcp, g.ycap);
    const uint32_t pad2 = zslice | (zslice << 16);      // both slots at the spare -inf

    // offsets (from the start of the slice, 16 bits each) of the target logits of this lane's two slots of every step:
    // requested first of all, they travel while the rest of the set-up runs
    uint32_t gor[NST > 0 ? NST : 1];
    if (warp < kSW && NST > 0) {
        const uint32_t* gt = reinterpret_cast<const uint32_t*>(g.goff + w_gstart);
        const int npairs = ((w_kcp + 63) & ~63) >> 1;       // pairs tabulated for this segment
#pragma unroll
        for (int st = 0; st < (NST > 0 ? NST : 1); ++st) {
            const int q = st * 32 + lane;
            uint32_t o = q < npairs ? __ldg(gt + q) : pad2;
            if (2 * q >= w_kcs) o = (o & 0xffff0000u) | zslice;            // beyond the cache: uncached route
            if (2 * q + 1 >= w_kcs) o = (o & 0x0000ffffu) | (zslice << 16);
            gor[st] = o;
        }
    } else {
        gor[0] = 0u;
    }

    // ---- state of the load warp's ring (used by its prologue here and by its loop below) ----------------------
    const int j0c = (int)min((long long)crank * kSW * g.Lw, (long long)P.N);
    const int lenc = max(0, min(P.N - j0c, kSW * g.Lw));
    const int lenc_v = lenc & ~(kZPer - 1);
    const uint32_t zbytes = (uint32_t)lenc_v * (uint32_t)sizeof(TZ);
    const uint32_t kbytes = lane < kSW ? (uint32_t)min(sd.y, g.ycap) * (uint32_t)sizeof(TY) : 0u;
    const uintptr_t y_end16 = reinterpret_cast<uintptr_t>(static_cast<const TY*>(P.drafter) +
                                                          (long long)(P.rows - 1) * P.drafter_stride + P.n) & ~uintptr_t(15);
    const TZ* nz = static_cast<const TZ*>(P.target) + (long long)grp * P.target_stride + j0c;
    const TY* ny = static_cast<const TY*>(P.drafter) + (long long)grp * P.drafter_stride + sd.x;
    const uint32_t l_yw_off = zslice + 16u + (uint32_t)(lane & (kSW - 1)) * (uint32_t)g.ystage;
    int l_s = 0;
    uint32_t l_eph = 1, l_st_a = dsm_a, l_fb = full_a, l_eb = empty_a;    // a fresh stage counts as released
    unsigned char* l_st_p = dsm;
    // one row: one bulk copy of the CTA's slice of the target row and one per warp of the matching drafter values,
    // into the stage the streaming warps have released
    auto load_row = [&]() {
        mbar_wait(l_eb, l_eph, &fail, spin_limit);
        // the few elements a 16-byte copy cannot cover go by plain stores: a slice that ends inside a
        // vector, and the very end of the drafter buffer
        const uintptr_t b0 = reinterpret_cast<uintptr_t>(ny), b1 = b0 + kbytes;
        const uintptr_t a0 = b0 & ~uintptr_t(15);
        uintptr_t a1 = (b1 + 15) & ~uintptr_t(15);
        if (a1 > y_end16) a1 = y_end16 > a0 ? y_end16 : a0;     // never read past the drafter buffer
        const uint32_t ybytes = kbytes ? (uint32_t)(a1 - a0) : 0u;
        if (lane < lenc - lenc_v) reinterpret_cast<TZ*>(l_st_p)[lenc_v + lane] = nz[lenc_v + lane];
        if (kbytes && a1 < b1) {
            const uintptr_t t0 = a1 > b0 ? a1 : b0;
            const int nt = (int)((b1 - t0) / sizeof(TY));
            for (int k = 0; k < nt; ++k) reinterpret_cast<TY*>(l_st_p + l_yw_off + (t0 - a0))[k] = reinterpret_cast<const TY*>(t0)[k];
        }
        const uint32_t total = zbytes + __reduce_add_sync(0xffffffffu, ybytes);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stage was last touched by plain loads and stores
        if (lane == 0) {
            if (total == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(l_fb) : "memory");
            else asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(l_fb), "r"(total) : "memory");
            for (uint32_t off = 0; off < zbytes; off += 32768u) {
                const uint32_t sz = min(32768u, zbytes - off);
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(l_st_a + off), "l"(reinterpret_cast<const char*>(nz) + off), "r"(sz), "r"(l_fb) : "memory");
            }
        }
        __syncwarp();
        if (ybytes)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(l_st_a + l_yw_off), "l"(a0), "r"(ybytes), "r"(l_fb) : "memory");
        nz += (long long)g.G * P.target_stride; ny += (long long)g.G * P.drafter_stride;
        l_st_a += stage; l_st_p += stage; l_fb += 8u; l_eb += 8u;
        if (++l_s == g.NS) { l_s = 0; l_eph ^= 1u; l_st_a = dsm_a; l_st_p = dsm; l_fb = full_a; l_eb = empty_a; }
    };
    // The load warp sets up the ring by itself and starts the first rows' copies right away, so that HBM's first
    // answer travels while the rest of the CTA is still setting up: it initialises the ring's barriers, gives the
    // parts of the target slices that no copy writes the weight 0 (beyond the vocabulary, and the 16 spare bytes of
    // every stage that padded gathers point at), and issues the first row.  The drafter regions need no such
    // care: every slot a copy did not fill (or filled with a neighbouring segment's values) is masked where it is read.
    const int pre_rows = min(1, rows_g);     // a single warp takes about 0.6 us to issue a row: the others follow the barrier
    if (warp == kWLoad) {
        if (lane == 0) {
            for (int k = 0; k < g.NS; ++k) {
                asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full_a + 8u * k));
                asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty_a + 8u * k), "r"(kSW));
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        {
            const uint32_t ninf16 = sizeof(TZ) == 2 ? 0xff80ff80u : 0xff800000u;      // -inf
            const uint32_t z0 = zbytes, z1 = zslice + 16u;        // [end of the copied vectors, spare bytes included)
            for (int k = 0; k < g.NS; ++k) {
                const uint32_t base = dsm_a + (uint32_t)k * stage;
#pragma unroll 8
                for (uint32_t o = z0 + 16u * lane; o < z1; o += 512u)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + o), "r"(ninf16) : "memory");
            }
        }
        __syncwarp();
        asm volatile("griddepcontrol.wait;" ::: "memory");     // the inputs may be the previous kernel's outputs
        for (int k = 0; k < pre_rows; ++k) load_row();
    }

    if (NST == 0 && warp < kSW) {          // the route with runtime loops keeps the offsets in shared memory
        const uint32_t* gt = reinterpret_cast<const uint32_t*>(g.goff + w_gstart);
        const int npairs = ((w_kcp + 63) & ~63) >> 1;
        const uint32_t gbase = dsm_a + off_goff + (uint32_t)warp * (uint32_t)g.ycap * 2u;
        for (int q = lane; q < nst * 32; q += 32) {
            uint32_t o = q < npairs ? __ldg(gt + q) : pad2;
            if (2 * q >= w_kcs) o = (o & 0xffff0000u) | zslice;
            if (2 * q + 1 >= w_kcs) o = (o & 0x0000ffffu) | (zslice << 16);
            sts32(gbase + (uint32_t)q * 4u, o);
        }
    }

    if (kTmem && warp == 0) {
        // all 512 columns: one CTA per SM (a kernel that asks for tensor memory on the same SM waits until this
        // one has given it back)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();                        // barriers initialised, padding and tables in place, tensor memory allocated
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    if (warp < kSW) {
        // ================================ streaming warps ============================================
        const int r0 = w_r0, kcp = w_kcp, kcs = w_kcs;
        const int j0 = (int)min((long long)seg * g.Lw, (long long)P.N);
        const bool ovf = kcp > kcs;
        const uint32_t zw_off = (uint32_t)warp * (uint32_t)g.Lw * (uint32_t)sizeof(TZ);
        const uint32_t yw_off = zslice + 16u + (uint32_t)warp * (uint32_t)g.ystage;
        const uint32_t csz = (uint32_t)g.ycap * 8u;
        const uint32_t cb0 = dsm_a + off_cache + (uint32_t)warp * (uint32_t)nb * csz + (uint32_t)lane * 16u;
        // tensor memory: this warp's quarter of the lanes (warp % 4), its 128 columns there, 4 columns per step and live row
        const uint32_t tb0 = tmem_base_s + ((uint32_t)(warp & 3) << 21) + (uint32_t)(warp >> 2) * (uint32_t)kTmemWarpCols;
        constexpr int kRowCols = 4 * (NST > 0 ? NST : 1);
        const uint32_t gl = dsm_a + off_goff + (uint32_t)warp * (uint32_t)g.ycap * 2u + (uint32_t)lane * 4u;
        // slot il = 64 st + 2 lane + h of the pair grid holds a kept token of the segment iff il < kcs, and
        // il > 0 or slot 0 is not the previous segment's; lim > 64 st + h says the first
        const int lim = kcs - 2 * lane;
        const bool last_step = NST > 1 && kcs > (NST - 1) * 64;      // the last of the NST steps holds slots of this warp
        const bool skip0 = w_dummy && lane == 0;
        const long long ystep = (long long)g.G * P.drafter_stride;
        const float2 l2e = splat(kLog2e);

        // ---- second visit of a row: sum of min(p, q~) over the cached kept tokens ----------------------
        // sv_sum: this lane's share, once the row's scalars are in place (par = row mod NB)
        auto sv_sum = [&](int itb, int par) -> float {
            const float theta = scal[par][4];
            const float2 f = fzy[par][warp];                  // p = f.x e_z,  q' = f.y e_y
            // q~ = q' + x (theta - q'),  x = p / N
            const float2 fz2 = splat(f.x), fy2 = splat(f.y), xs2 = splat(f.x * inv_n), th2 = splat(theta), neg1 = splat(-1.f);
            float2 ak2 = splat(0.f);
            const uint32_t cb = cb0 + (uint32_t)par * csz;
            auto sv_math = [&](uint4 c4) {
                const float2 ez = make_float2(__uint_as_float(c4.x), __uint_as_float(c4.y));
                const float2 ey = make_float2(__uint_as_float(c4.z), __uint_as_float(c4.w));
                const float2 p = fmul2(ez, fz2), qp = fmul2(ey, fy2), x = fmul2(ez, xs2);
                const float2 w = ffma2(x, ffma2(qp, neg1, th2), qp);
                ak2 = fadd2(ak2, make_float2(fminf(p.x, w.x), fminf(p.y, w.y)));
            };
            if (NST > 0) {
                // all loads first (tensor memory answers asynchronously), then the arithmetic
                uint4 c4[NST > 0 ? NST : 1];
#pragma unroll
                for (int st = 0; st < (NST > 0 ? NST : 1); ++st)
                    if (st < NST - 1 || NST == 1 || last_step) c4[st] = tmem_ld4(tb0 + (uint32_t)(par * kRowCols + st * 4));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int st = 0; st < (NST > 0 ? NST : 1); ++st)
                    if (st < NST - 1 || NST == 1 || last_step) sv_math(c4[st]);
            } else {
#pragma unroll 2
                for (int st = 0; st < nst; ++st) sv_math(lds128(cb + (uint32_t)st * 512u));
            }
            float ak = ak2.x + ak2.y;
            if (ovf) {   // kept tokens beyond the cache: from global memory again
                const long long row = grp + (long long)itb * g.G;
                const TZ* zrow = static_cast<const TZ*>(P.target) + row * P.target_stride;
                const TY* yrow = static_cast<const TY*>(P.drafter) + row * P.drafter_stride;
                const float m_w = wrec[par][warp][4], my_w = wrec[par][warp][5];
                const float zoff = m_w > -INFINITY ? -m_w * kLog2e : 0.f, yoff = my_w > -INFINITY ? -my_w * kLog2e : 0.f;
                for (int il = kcs + lane; il < kcp; il += 32) {
                    const float ez = ex2(fmaf(to_float<TZ>(zrow[__ldg(P.ids + r0 + il)]), kLog2e, zoff));
                    const float y = to_float<TY>(yrow[r0 + il]);
                    const float ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff)) : y;
                    const float p = ez * f.x, qp = ey * f.y;
                    ak += fminf(p, fmaf(p * inv_n, theta - qp, qp));
                }
            }
            return ak;
        };
        auto sv_finish = [&](int par, float ak) {
            ak = warp_sum(ak);
            if (lane == 0) {
                akv[par][warp] = ak;
                mbar_arrive(smem_u32(&bbar[par]));
            }
        };

        // ---- main loop: first visit of row it, second visit of row it - (NB - 1) -----------------------
        const TY* cy = static_cast<const TY*>(P.drafter) + (long long)grp * P.drafter_stride + r0;   // slot 0 of the current row
        int s = 0;
        uint32_t sph = 0, st_a = dsm_a, fb = full_a, eb = empty_a;
        int par = 0;                                     // it mod NB
        int bit = 0, bpar = 0;                           // next row to get its second visit, the same mod NB
        uint32_t bph = 0;
        auto first_visit = [&]() {
            const uint32_t zs_a = st_a + zw_off;
            const uint32_t shb = (uint32_t)(reinterpret_cast<uintptr_t>(cy) & 15u);      // slot 0 sits this many bytes into the warp's region
            const uint32_t ysb_a = st_a + yw_off + shb;                                      // slot 0 of the warp's pair grid
            const uint32_t ys_a = ysb_a + (uint32_t)lane * 2u * (uint32_t)sizeof(TY);           // this lane's pair of step 0

            // maximum of the segment (the scale of its exponentials)
            uint4 zv[NIT > 0 ? NIT : 1];
            MaxAcc<TZ> mz;
            if (NIT > 0) {
#pragma unroll
                for (int k = 0; k < (NIT > 0 ? NIT : 1); ++k) zv[k] = lds128(zs_a + (uint32_t)(k * 32 + lane) * 16u);
#pragma unroll
                for (int k = 0; k < (NIT > 0 ? NIT : 1); ++k) mz.push(zv[k]);
            } else {
#pragma unroll 4
                for (int t = lane * kZPer; t < g.Lw; t += 32 * kZPer) mz.push(lds128(zs_a + (uint32_t)t * (uint32_t)sizeof(TZ)));
            }
            // Scale of the drafter exponentials: not the maximum of the warp's kept values (finding it first
            // would hold up every exponential) but one of them, the first; any scale gives the same result
            // as long as nothing grows too large, which the sum found along the way confirms below.
            float my_w = KIND == RDK_LOGITS ? -INFINITY : 0.f;
            if (KIND == RDK_LOGITS && kcp > w_dummy)
                my_w = kcs > w_dummy ? lds_z<TY>(ysb_a + (uint32_t)w_dummy * (uint32_t)sizeof(TY)) : to_float<TY>(cy[w_dummy]);
            const float m_w = warp_max_redux(mz.result());
            const float zoff = m_w > -INFINITY ? -m_w * kLog2e : 0.f;
            float yoff = my_w > -INFINITY ? -my_w * kLog2e : 0.f;

            // soft-max sweep: sum of e over the segment
            float2 Ea = splat(0.f), Eb = splat(0.f);
            {
                const float2 of = splat(zoff);
                if (NIT > 0) {
#pragma unroll
                    for (int k = 0; k < (NIT > 0 ? NIT : 1); ++k) exp_sum_vec<TZ>(zv[k], l2e, of, Ea, Eb);
                } else {
#pragma unroll 4
                    for (int t = lane * kZPer; t < g.Lw; t += 32 * kZPer)
                        exp_sum_vec<TZ>(lds128(zs_a + (uint32_t)t * (uint32_t)sizeof(TZ)), l2e, of, Ea, Eb);
                }
            }
            // kept tokens: e_z, e_y, their sums; the pairs go to the cache
            float K1s, Zqs, ths;
            const uint32_t cbA = cb0 + (uint32_t)par * csz;
            auto kept_step = [&](int st, uint32_t go, float2 zof, float2 yof, float2& K1, float2& Zq, float2& th) {
                const float2 z = make_float2(lds_z<TZ>(st_a + (go & 0xffffu)), lds_z<TZ>(st_a + (go >> 16)));
                const float2 y = lds_ypair<TY>(ys_a + (uint32_t)st * 64u * (uint32_t)sizeof(TY));
                const bool v0 = (lim > st * 64) && !(st == 0 && skip0), v1 = lim > st * 64 + 1;
                const float2 ez = ex2_2(ffma2(z, l2e, zof));
                float2 ey;
                if (KIND == RDK_LOGITS) {
                    float2 t = ffma2(y, l2e, yof);
                    t.x = v0 ? t.x : -INFINITY; t.y = v1 ? t.y : -INFINITY;
                    ey = ex2_2(t);
                } else {
                    ey = make_float2(v0 ? y.x : 0.f, v1 ? y.y : 0.f);
                }
                K1 = fadd2(K1, ez); Zq = fadd2(Zq, ey); th = ffma2(ez, ey, th);
                if (kTmem) tmem_st4(tb0 + (uint32_t)(par * kRowCols + st * 4), ez.x, ez.y, ey.x, ey.y);
                else sts128(cbA + (uint32_t)st * 512u, ez.x, ez.y, ey.x, ey.y);
            };
            auto kept_pass = [&]() {
                float2 K1 = splat(0.f), Zq = splat(0.f), th = splat(0.f);
                const float2 zof = splat(zoff), yof = splat(yoff);
                if (NST > 0) {
#pragma unroll
                    for (int st = 0; st < (NST > 0 ? NST : 1); ++st)
                        if (st < NST - 1 || NST == 1 || last_step) kept_step(st, gor[st], zof, yof, K1, Zq, th);
                } else {
#pragma unroll 2
                    for (int st = 0; st < nst; ++st) kept_step(st, lds32(gl + (uint32_t)st * 128u), zof, yof, K1, Zq, th);
                }
                K1s = K1.x + K1.y; Zqs = Zq.x + Zq.y; ths = th.x + th.y;
                if (kTmem) asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                if (ovf) {
                    for (int il = kcs + lane; il < kcp; il += 32) {               // kept tokens beyond the cache
                        const float ez = ex2(fmaf(lds_z<TZ>(zs_a + (uint32_t)(__ldg(P.ids + r0 + il) - j0) * (uint32_t)sizeof(TZ)), kLog2e, zoff));
                        const float y = to_float<TY>(cy[il]);
                        const float ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff)) : y;
                        K1s += ez; Zqs += ey; ths = fmaf(ez, ey, ths);
                    }
                }
            };
            kept_pass();
            if (KIND == RDK_LOGITS) {
                // 2^64 and beyond (or not a number), or the first value was -inf: a poor scale, take the maximum
                const bool poor = kcp > w_dummy && !(my_w > -INFINITY);
                if (poor || __any_sync(0xffffffffu, !(Zqs < 1.8e19f))) {
                    float ym = -INFINITY;
                    for (int st = 0; st < nst; ++st) {
                        const float2 y = lds_ypair<TY>(ys_a + (uint32_t)st * 64u * (uint32_t)sizeof(TY));
                        const bool v0 = (lim > st * 64) && !(st == 0 && skip0), v1 = lim > st * 64 + 1;
                        ym = fmaxf(ym, fmaxf(v0 ? y.x : -INFINITY, v1 ? y.y : -INFINITY));
                    }
                    if (ovf) for (int il = kcs + lane; il < kcp; il += 32) ym = fmaxf(ym, to_float<TY>(cy[il]));
                    my_w = warp_max_redux(ym);
                    yoff = my_w > -INFINITY ? -my_w * kLog2e : 0.f;
                    kept_pass();
                }
            }
            const float E1s = (Ea.x + Ea.y) + (Eb.x + Eb.y);
            const float tot = warp_sum4(E1s, K1s, Zqs, ths, lane);      // lanes 0, 8, 16, 24 hold the four totals
            // the warp's record goes to the publish warp, the stage back to the load warp
            if ((lane & 7) == 0) wrec[par][warp][lane >> 3] = tot;
            if (lane == 0) *reinterpret_cast<float2*>(&wrec[par][warp][4]) = make_float2(m_w, my_w);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&abar[par]));
                mbar_arrive(eb);
            }
        };
        for (int it = 0; it < rows_g; ++it) {
            mbar_wait(fb, sph, &fail, spin_limit);
            first_visit();
            if (it >= defer) {
                mbar_wait(smem_u32(&rbar[bpar]), bph, &fail, spin_limit);
                sv_finish(bpar, sv_sum(bit, bpar));
                ++bit;
                if (++bpar == nb) { bpar = 0; bph ^= 1u; }
            }
            if (++par == nb) par = 0;
            cy += ystep;
            st_a += stage; fb += 8u; eb += 8u;
            if (++s == g.NS) { s = 0; sph ^= 1u; st_a = dsm_a; fb = full_a; eb = empty_a; }
        }
        for (; bit < rows_g; ++bit) {
            mbar_wait(smem_u32(&rbar[bpar]), bph, &fail, spin_limit);
            sv_finish(bpar, sv_sum(bit, bpar));
            if (++bpar == nb) { bpar = 0; bph ^= 1u; }
        }
    } else if (warp == kWPublish) {
        // ================================ publish warp ==================================================
        // Per row: fold the CTA's 16 warp records into one and publish it in global memory; NB rows
        // later, when the second visits of the row are over, write its per-segment sums for the draw
        // kernel.  Lane w < 16 looks after warp w; what later steps need of a row is parked in
        // pend[row mod 16].
        // This grid may have been started while the previous kernel of the stream was draining: nothing
        // of the workspace and none of the inputs is touched before that kernel is complete.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        auto finish_row = [&](int itf) {
            const int pf = itf % nb;
            const long long row = grp + (long long)itf * g.G;
            mbar_wait(smem_u32(&bbar[pf]), (uint32_t)((itf / nb) & 1), &fail, spin_limit);
            float* rec = P.rec + row * kRecFloats;
            if (lane < kSW) {
                const float4 w0 = *reinterpret_cast<const float4*>(&pend[itf & 15][lane][0]);
                const float4 f4 = *reinterpret_cast<const float4*>(&pend[itf & 15][lane][4]);     // fz, fy, theta, a row scalar (from the collect warp)
                const float theta = f4.z, ak = akv[pf][lane];
                // sums over the segment: p; w of the not-kept tokens (theta x); w of the kept tokens from the moments
                const float segP = w0.x * f4.x;
                const float xs = f4.x * inv_n;
                const float oov = theta * xs * fmaxf(0.f, w0.x - w0.y);
                const float Kw = f4.y * w0.z - f4.y * xs * w0.w + theta * xs * w0.y;
                const float a_s = oov + ak;
                reinterpret_cast<float4*>(rec + 16)[seg] = make_float4(oov + Kw, a_s, fmaxf(0.f, segP - a_s), segP);
                if (crank == 0 && lane < 5) rec[lane] = lane == 4 ? theta : f4.w;     // -m log2e, 1/Zp, -my log2e, 1/Zq, theta
            }
        };
        for (int it = 0; it < rows_g + nb; ++it) {
            if (it < rows_g) {
                const int par = it % nb;
                const long long row = grp + (long long)it * g.G;
                mbar_wait(smem_u32(&abar[par]), (uint32_t)((it / nb) & 1), &fail, spin_limit);
                float E1 = 0.f, Zq = 0.f, th = 0.f, m = -INFINITY, my = -INFINITY, K1 = 0.f;
                if (lane < kSW) {
                    const volatile float* wr = &wrec[par][lane][0];
                    E1 = wr[0]; K1 = wr[1]; Zq = wr[2]; th = wr[3]; m = wr[4]; my = wr[5];
                    *reinterpret_cast<float4*>(&pend[it & 15][lane][0]) = make_float4(E1, K1, Zq, th);
                    *reinterpret_cast<float2*>(&pend[it & 15][lane][4]) = make_float2(m, my);     // the warp's maxima, until the factors replace them
                }
                combine_records(E1, Zq, th, m, my, lane);
                {
                    // five (value, tag) words, one per lane
                    const float v = lane == 0 ? E1 : (lane == 1 ? Zq : (lane == 2 ? th : (lane == 3 ? m : my)));
                    if (lane < 5) st_tagged(P.xrec + ((size_t)row * g.C + crank) * kXrecBytes + 8 * lane, v, g.tag);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&pbar[it & 15]));
            }
            if (it - nb >= 0) finish_row(it - nb);
        }
    } else if (warp == kWCollect) {
        // ================================ collect warp ==================================================
        // Per row: gather the C records of the row from global memory, leave the row scalars and every
        // warp's factors in shared memory for the second visits.
        asm volatile("griddepcontrol.wait;" ::: "memory");     // see the publish warp
        for (int it = 0; it < rows_g; ++it) {
            const int pc = it % nb;
            const long long row = grp + (long long)it * g.G;
            float E1 = 0.f, Zq = 0.f, th = 0.f, m = -INFINITY, my = -INFINITY;
            if (lane < g.C) {
                const unsigned char* xr = P.xrec + ((size_t)row * g.C + lane) * kXrecBytes;
                unsigned long long w[5];
                unsigned spins = 0;
                for (;;) {
                    bool ok = true;
#pragma unroll
                    for (int k = 0; k < 5; ++k) w[k] = ld_tagged(xr + 8 * k);
#pragma unroll
                    for (int k = 0; k < 5; ++k) ok = ok && (uint32_t)(w[k] >> 32) == g.tag;
                    if (ok) break;
                    if (++spins > spin_limit || ld_volatile_s32(&fail)) { atomicExch(&fail, 1); break; }
                    __nanosleep(20);
                }
                E1 = __uint_as_float((uint32_t)w[0]); Zq = __uint_as_float((uint32_t)w[1]); th = __uint_as_float((uint32_t)w[2]);
                m = __uint_as_float((uint32_t)w[3]); my = __uint_as_float((uint32_t)w[4]);
            }
            combine_records(E1, Zq, th, m, my, lane);
            const float inv_zp = 1.f / E1, inv_zq = 1.f / Zq;
            const float theta = th * inv_zp * inv_zq;
            mbar_wait(smem_u32(&pbar[it & 15]), (uint32_t)((it >> 4) & 1), &fail, spin_limit);     // this CTA's own record of the row is parked
            if (lane < kSW) {
                const float2 mw = *reinterpret_cast<const float2*>(&pend[it & 15][lane][4]);
                float2 f;
                f.x = (mw.x > -INFINITY ? ex2((mw.x - m) * kLog2e) : 0.f) * inv_zp;
                f.y = (KIND == RDK_LOGITS ? (mw.y > -INFINITY ? ex2((mw.y - my) * kLog2e) : 0.f) : 1.f) * inv_zq;
                fzy[pc][lane] = f;
                // lanes 0..3 also carry the row scalars the draws need: -m log2e, 1/Zp, -my log2e, 1/Zq
                const float sc = lane == 0 ? -m * kLog2e : (lane == 1 ? inv_zp : (lane == 2 ? (KIND == RDK_LOGITS ? -my * kLog2e : 0.f) : inv_zq));
                *reinterpret_cast<float4*>(&pend[it & 15][lane][4]) = make_float4(f.x, f.y, theta, sc);
            }
            if (lane == 0) scal[pc][4] = theta;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&rbar[pc]));
            if (crank == 0 && P.counters && row % P.positions == 0)
                for (int t = lane; t < P.trials; t += 32) P.counters[(row / P.positions) * P.trials + t] = 0;
        }
    } else {
        // ================================ load warp =====================================================
        // the first row went out during the set-up; one row per stage as the streaming warps release them
        for (int it = pre_rows; it < rows_g; ++it) load_row();
        if (ld_volatile_s32(&fail)) {
            // A wait gave up somewhere, so nobody may have waited for the last copies: let them land before
            // the CTA leaves (bounded as well, on a count of its own).
            for (int k = 0; k < g.NS && k < rows_g; ++k) {
                const int last_it = ((rows_g - 1 - k) / g.NS) * g.NS + k;        // last row that used stage k
                const uint32_t bar = full_a + 8u * (uint32_t)k, parity = (uint32_t)((last_it / g.NS) & 1);
                uint32_t done = 0;
                for (unsigned spins = 0; !done && spins < (1u << 16); ++spins) {
                    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
                    if (!done) __nanosleep(100);
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (kTmem && warp == 0) {               // every path ends here, also after a wait that gave up
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "r"(kTmemCols) : "memory");
    }
    if (tid == 0 && fail && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_TIMEOUT);
}

__device__ __forceinline__ bool index_matches(const RowParams& P) {
    return P.header[kHdrMagic] == kIdxMagic && P.header[kHdrN] == P.N && P.header[kHdrn] == P.n;
}

// ------------------------------------------------------------------------------------------------
// kernel 2: one CTA per (row, trial) turns the row's record into draws
// ------------------------------------------------------------------------------------------------
// DT threads per CTA: half of the warps work on the draft draw, half on the residual draw.
template <typename TZ, typename TY, int KIND, int DT>
__global__ void __launch_bounds__(DT)
rdk_draw_kernel(const RowParams P, const int nseg, const int Lw) {
    __shared__ double cdfW[kMaxSeg], cdfR[kMaxSeg], cdfP[kMaxSeg];
    __shared__ float sums[2][kMaxChunks];
    __shared__ float alpha_s;
    __shared__ int res_tok[2];
    __shared__ float res_p[2], res_w[2];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x / P.trials, t = blockIdx.x % P.trials;
    const float* rec = P.rec + (long long)row * kRecFloats;
    DrawCtx d;
    if (!index_matches(P)) return;                 // kernel 1 has reported it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a following stream kernel may set itself up meanwhile
    asm volatile("griddepcontrol.wait;" ::: "memory");   // kernel 1 (launched just before) is complete and visible; so is
                                                         // whatever produced this call's inputs
    const float* u = P.uniforms + ((long long)row * P.trials + t) * 4;
    const float u0 = __ldg(u), u1 = __ldg(u + 1), u2 = __ldg(u + 2);
    d.c.offg = __ldcg(rec + kRecOffg); d.c.inv_zp = __ldcg(rec + kRecInvZp); d.c.yoffg = __ldcg(rec + kRecYoffg);
    d.c.inv_zq = __ldcg(rec + kRecInvZq); d.c.theta = __ldcg(rec + kRecTheta); d.c.inv_n = 1.f / (float)P.N;
    d.c.inv_s = 1.f;

    if (warp < 3) {   // fp64 prefix sums over the segments: warp 0 those of w, warp 1 of max(0, p - q~), warp 2 of p
        double* cdf = warp == 0 ? cdfW : (warp == 1 ? cdfR : cdfP);
        // a lane takes K consecutive segments (all loads first), sums them up in order, and one scan over
        // the lanes' totals places its run
        constexpr int K = kMaxSeg / 32;
        const int per = (nseg + 31) >> 5, s0 = lane * per;
        float v[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            v[k] = 0.f;
            if (k < per && s0 + k < nseg) {
                const float4 r4 = __ldcg(reinterpret_cast<const float4*>(rec + 16) + s0 + k);
                v[k] = warp == 0 ? r4.x : (warp == 1 ? r4.z : r4.w);
            }
        }
        double run[K], x = 0.0;
#pragma unroll
        for (int k = 0; k < K; ++k) { x += (double)v[k]; run[k] = x; }
        double incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double a = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += a;
        }
        double before = __shfl_up_sync(0xffffffffu, incl, 1);      // the previous lane's last value, so the sequence never steps back
        if (lane == 0) before = 0.0;
#pragma unroll
        for (int k = 0; k < K; ++k)
            if (k < per && s0 + k < nseg) cdf[s0 + k] = before + run[k];
    } else if (warp == 3) {   // alpha = sum over the segments of sum min(p, q~)
        float alpha_l = 0.f;
        for (int s = lane; s < nseg; s += 32) alpha_l += __ldcg(reinterpret_cast<const float4*>(rec + 16) + s).y;
        alpha_l = warp_sum(alpha_l);
        if (lane == 0) alpha_s = alpha_l;
    }
    __syncthreads();
    const double S_d = cdfW[nseg - 1], R_d = cdfR[nseg - 1], Pt_d = cdfP[nseg - 1];
    if (t == 0 && tid == 0) {
        if (P.alpha) P.alpha[row] = alpha_s;
        if (P.theta) P.theta[row] = d.c.theta;
        if (P.S) P.S[row] = (float)S_d;
        if (P.residual_mass) P.residual_mass[row] = (float)R_d;
    }
    const TZ* zrow = static_cast<const TZ*>(P.target) + (long long)row * P.target_stride;
    d.zrow = zrow; d.yrow = static_cast<const TY*>(P.drafter) + (long long)row * P.drafter_stride;
    d.zvec = (reinterpret_cast<uintptr_t>(zrow) & 15u) == 0;
    d.mask = P.mask; d.rank = P.rank; d.N = P.N;

    // group 0 (first half of the warps): the draft draw from w; group 1: the residual draw, computed
    // alongside (it is only used if the draft is rejected)
    constexpr int kGW = DT / 64;             // warps per group
    const int g = warp / kGW, wg = warp % kGW;
    const bool from_p = !(R_d > 0.0);                 // p and q~ coincide: the replacement comes from p itself
    const double* cdf = g == 0 ? cdfW : (from_p ? cdfP : cdfR);
    const int what = g == 0 ? kPickW : (from_p ? kPickP : kPickR);
    const double thr = g == 0 ? (double)u0 * S_d : (double)u2 * (from_p ? Pt_d : R_d);
    const int seg = min(first_above(cdf, nseg, thr), nseg - 1);
    const float rem = (float)(thr - (seg ? cdf[seg - 1] : 0.0));
    const int seg_lo = (int)min((long long)seg * Lw, (long long)P.N);
    const int seg_end = (int)min((long long)P.N, (long long)seg_lo + Lw);
    const int nch = (Lw + kSeg - 1) / kSeg;
    float p[kVec], w[kVec], x[kVec];          // of the last chunk this warp summed
    for (int ch = wg; ch < nch; ch += kGW) {
        draw_x<TZ, TY, KIND>(d, what, seg_lo + ch * kSeg + lane * kVec, seg_end, p, w, x);
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < kVec; ++k) s += x[k];
        s = warp_sum(s);
        if (lane == 0) sums[g][ch] = s;
    }
    __syncthreads();
    {   // every warp finds the chunk of its group; the warp that owns it picks the token
        float cum = 0.f, before = 0.f;
        int chosen = -1, last_pos = -1;
        for (int ch = 0; ch < nch; ++ch) {
            const float s = sums[g][ch];
            if (s > 0.f) {
                if (chosen < 0 && cum + s > rem) { chosen = ch; before = cum; }
                last_pos = ch;
                cum += s;
            }
        }
        float r_in = rem - before;
        if (chosen < 0) { chosen = last_pos; r_in = INFINITY; }      // rounding: the last positive token
        if (chosen < 0) {
            if (wg == 0 && lane == 0) { res_tok[g] = seg_lo; res_p[g] = 0.f; res_w[g] = 0.f; }
        } else if (chosen % kGW == wg) {
            // the chunk is still in this warp's registers unless the warp went on to a later one
            if (chosen + kGW < nch) draw_x<TZ, TY, KIND>(d, what, seg_lo + chosen * kSeg + lane * kVec, seg_end, p, w, x);
            int sel = pick_in_segment(x, r_in, lane);
            if (sel < 0) sel = 0;
            float ps = 0.f, ws = 0.f;
#pragma unroll
            for (int k = 0; k < kVec; ++k) if (k == (sel & (kVec - 1))) { ps = p[k]; ws = w[k]; }
            ps = __shfl_sync(0xffffffffu, ps, sel / kVec);
            ws = __shfl_sync(0xffffffffu, ws, sel / kVec);
            if (lane == 0) { res_tok[g] = seg_lo + chosen * kSeg + sel; res_p[g] = ps; res_w[g] = ws; }
        }
    }
    __syncthreads();
    // The records that the CTAs of a group exchanged for this row are spent: wipe them, tags included.
    // The launches of a replayed graph carry the same tag every time and must not meet their old records.
    if (t == 0 && tid >= 64 && tid - 64 < (nseg / kSW) * (kXrecBytes / 16))
        __stcg(reinterpret_cast<uint4*>(P.xrec + (size_t)row * (size_t)(nseg / kSW) * kXrecBytes) + (tid - 64), make_uint4(0u, 0u, 0u, 0u));
    if (tid == 0) {
        const int dtok = res_tok[0];
        const float pd = res_p[0], qd = res_w[0] * d.c.inv_s;
        const float a_prob = (pd >= qd) ? 1.f : pd / qd;
        const bool acc = u1 * qd < pd;
        const long long o = (long long)row * P.trials + t;
        if (P.draft_token) P.draft_token[o] = dtok;
        if (P.accepted) P.accepted[o] = acc ? 1 : 0;
        if (P.accept_prob) P.accept_prob[o] = a_prob;
        if (P.out_token) P.out_token[o] = acc ? dtok : res_tok[1];
        if (P.accepted_len && P.accepted && P.counters) {
            // the last position of a sequence to finish counts the accepted prefix (Algorithm 4 step 7)
            const int b = row / P.positions;
            __threadfence();
            const int old = atomicAdd(P.counters + b * P.trials + t, 1);
            if (old == P.positions - 1) {
                __threadfence();
                int k = 0;
                const volatile uint8_t* af = P.accepted;
                while (k < P.positions && af[((long long)b * P.positions + k) * P.trials + t]) ++k;
                P.accepted_len[b * P.trials + t] = k;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
static int fast_steps(const StreamGeo& g, int nit) {
    const int nst = g.ycap / 64;
    return (nit == kFastNit && nst >= 1 && nst <= kMaxFastSteps) ? nst : 0;
}

// offsets_in_smem = false is the unrolled route: offsets in registers and the pair cache in tensor memory
static size_t stream_smem(const StreamGeo& g, size_t es, bool offsets_in_smem) {
    const size_t stage = (size_t)kSW * g.Lw * es + 16 + (size_t)kSW * g.ystage;
    // + cache (8 bytes per slot and live row) and offsets (2 bytes per slot) where they live here, barriers
    return (size_t)g.NS * stage + (offsets_in_smem ? (size_t)kSW * g.ycap * (8 * g.NB + 2) : 0) + (size_t)g.NS * 16;
}

// Stage count, live rows and cache capacity for a vocabulary of N tokens with n kept ids; false when
// the shapes do not fit shared memory.
static bool plan_stream(int N, int n, size_t es, size_t ys, bool fast_types, StreamGeo& g) {
    const size_t budget = 212 * 1024;      // dynamic shared memory a CTA may ask for: 227 KB less the static part (14.2 KB)
    StreamSegs sg;
    if (!stream_segments(N, es, sg)) return false;
    g.C = sg.C; g.Lw = sg.Lw; g.nv = sg.nv;
    if ((g.Lw + kSeg - 1) / kSeg > kMaxChunks) return false;
    const long long expect = ((long long)n * g.Lw + N - 1) / N;
    long long cap = expect + expect / 8 + 32;
    const long long most = (long long)(n < g.Lw ? n : g.Lw) + 1;
    if (cap > most) cap = most;
    cap = (cap + 63) / 64 * 64;
    auto fits = [&](long long c) {
        g.ycap = (int)c;
        g.ystage = (int)((((size_t)c + 16) * ys + 15) & ~size_t(15));
        const bool in_regs = fast_types && fast_steps(g, g.nv) > 0;
        return stream_smem(g, es, !in_regs) <= budget;
    };
    // The exchange of a row between the CTAs of its group takes several microseconds (two round trips to L2
    // and the folding on either side), and a row holds its place in the pair cache for that long: the
    // second visit should trail by as many rows as there is room for.
    // Unrolled route: the pair cache is in tensor memory (128 columns per warp, 4 per step and live row), and
    // shared memory goes to the stages, of which more than the HBM latency needs are of no use.
    g.ycap = (int)cap;
    if (fast_types && fast_steps(g, g.nv) > 0) {
        const int nst = fast_steps(g, g.nv);
        g.NB = kTmemWarpCols / (4 * nst);
        if (g.NB > kMaxNB) g.NB = kMaxNB;
        for (g.NS = 4; g.NS >= 2; --g.NS)
            if (fits(cap)) return true;
    }
    // Otherwise the cache shares shared memory with the stages: prefer live rows over stages, then give up cache.
    static const int pref[][2] = {{4, 3}, {5, 2}, {4, 2}, {3, 3}, {3, 2}};     // {NB, NS}, by measured speed
    for (const auto& pr : pref) {
        g.NB = pr[0]; g.NS = pr[1];
        if (fits(cap)) return true;
    }
    for (long long c = cap - 64; c >= 64; c -= 64)
        if (fits(c)) return true;
    return false;
}

static std::atomic<unsigned> g_spin_limit{kSpinLimitDefault};

template <typename TZ, typename TY, int KIND, int NIT, int NST>
static cudaError_t launch_stream(const RowParams& P, StreamGeo g, cudaStream_t s) {
    auto kern = rdk_stream_kernel<TZ, TY, KIND, NIT, NST>;
    const size_t smem = stream_smem(g, sizeof(TZ), NST == 0);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // how many CTAs are resident at once (cached per kernel instance, shared-memory size and device)
    static thread_local int c_dev = -1, c_ctas = 0;
    static thread_local size_t c_smem = 0;
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev != c_dev || smem != c_smem) {
        int sms = 0, per_sm = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kSThreads, smem);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorNotSupported;
        c_dev = dev; c_smem = smem; c_ctas = sms * per_sm;
    }
    if (c_ctas < g.C) return cudaErrorNotSupported;
    g.G = c_ctas / g.C;
    if (g.G > P.rows) g.G = P.rows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(g.G * g.C), 1, 1);
    cfg.blockDim = dim3(kSThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    // The CTAs of a group wait for one another, so all of the grid must be resident together.  A cooperative launch
    // makes the driver guarantee that, at a price of about 4 us per launch.  It is asked for on the first launch of a
    // (kernel, device, shared-memory size) only: that launch proves that the grid fits the SMs this context may
    // use; later launches of the same shape are ordinary ones (one CTA per SM, grid <= the SM count), and should
    // something else keep CTAs from becoming resident, their peers' bounded waits end in RDK_ERR_TIMEOUT.
    static thread_local int v_dev = -1;
    static thread_local size_t v_smem = 0;
    const bool fits_proven = v_dev == dev && v_smem == smem;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may set itself up while the previous kernel drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    static std::atomic<int> c_pdl{1};                 // whether the two attributes are accepted together on this system
    const int with_pdl = c_pdl.load();
    if (fits_proven) {
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, P, g);
    } else {
        if (!with_pdl) { attr[0] = attr[1]; cfg.numAttrs = 1; } else cfg.numAttrs = 2;
        e = cudaLaunchKernelEx(&cfg, kern, P, g);
        if (with_pdl && (e == cudaErrorNotSupported || e == cudaErrorInvalidValue)) {
            (void)cudaGetLastError();
            attr[0] = attr[1]; cfg.numAttrs = 1;
            e = cudaLaunchKernelEx(&cfg, kern, P, g);
            if (e == cudaSuccess) c_pdl.store(0);     // the pair is what this system refuses
        }
        if (e == cudaSuccess) { v_dev = dev; v_smem = smem; }
    }
    if (e == cudaErrorCooperativeLaunchTooLarge) {   // fewer SMs at hand than the device reports: the one-CTA-per-row kernel serves
        (void)cudaGetLastError();
        return cudaErrorNotSupported;
    }
    if (e != cudaSuccess) return e;
    // small CTAs when the draws of all rows would not be resident at once with large ones (shorter
    // tail), large CTAs otherwise (shorter chain per row)
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const bool small_ctas = (long long)P.rows * P.trials > (long long)sms * 8;
    cudaLaunchConfig_t dcfg = {};
    dcfg.gridDim = dim3((unsigned)(P.rows * P.trials), 1, 1);
    dcfg.blockDim = dim3(small_ctas ? 128 : 256, 1, 1);
    dcfg.dynamicSmemBytes = 0;
    dcfg.stream = s;
    cudaLaunchAttribute dattr[1];
    dattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while kernel 1 drains
    dattr[0].val.programmaticStreamSerializationAllowed = 1;
    dcfg.attrs = dattr;
    dcfg.numAttrs = 1;
    if (small_ctas) return cudaLaunchKernelEx(&dcfg, rdk_draw_kernel<TZ, TY, KIND, 128>, P, g.C * kSW, g.Lw);
    return cudaLaunchKernelEx(&dcfg, rdk_draw_kernel<TZ, TY, KIND, 256>, P, g.C * kSW, g.Lw);
}

template <typename TZ, typename TY, int KIND>
static cudaError_t launch_nit(const RowParams& P, const StreamGeo& g, cudaStream_t s) {
    // the common segment length (four 16-byte vectors per lane) gets the register-resident sweep
    if (g.nv == kFastNit) return launch_stream<TZ, TY, KIND, kFastNit, 0>(P, g, s);
    return launch_stream<TZ, TY, KIND, 0, 0>(P, g, s);
}

template <typename TZ, typename TY>
static cudaError_t launch_kind_s(const RowParams& P, int kind, const StreamGeo& g, cudaStream_t s) {
    return kind == RDK_LOGITS ? launch_nit<TZ, TY, RDK_LOGITS>(P, g, s) : launch_nit<TZ, TY, RDK_PROBS>(P, g, s);
}

// bf16 logits on both sides with the common segment length: the kept-token passes unrolled
static cudaError_t launch_fast(const RowParams& P, const StreamGeo& g, int nst, cudaStream_t s) {
    using B = __nv_bfloat16;
    switch (nst) {
        case 1: return launch_stream<B, B, RDK_LOGITS, kFastNit, 1>(P, g, s);
        case 2: return launch_stream<B, B, RDK_LOGITS, kFastNit, 2>(P, g, s);
        case 3: return launch_stream<B, B, RDK_LOGITS, kFastNit, 3>(P, g, s);
        case 4: return launch_stream<B, B, RDK_LOGITS, kFastNit, 4>(P, g, s);
        case 5: return launch_stream<B, B, RDK_LOGITS, kFastNit, 5>(P, g, s);
        case 6: return launch_stream<B, B, RDK_LOGITS, kFastNit, 6>(P, g, s);
        default: return cudaErrorNotSupported;
    }
}

static size_t ws_off_counters(int rows) { return idx_align((size_t)rows * kRecFloats * sizeof(float)); }
static size_t ws_off_xrec(int rows, int batch, int trials) { return ws_off_counters(rows) + idx_align((size_t)batch * trials * sizeof(int32_t)); }

size_t stream_workspace_bytes(int rows, int batch, int trials) {
    return ws_off_xrec(rows, batch, trials) + idx_align((size_t)rows * kMaxGroup * kXrecBytes);
}

// A non-zero 32-bit value that differs from the one of every recent call of this process and that
// stale memory is unlikely to hold.  (The kernel wipes a call's records, so a captured call that
// is replayed with this same value starts from a workspace without them.)
static uint32_t next_tag() {
    static std::atomic<uint32_t> ctr{
        (uint32_t)std::chrono::high_resolution_clock::now().time_since_epoch().count() * 0x9E3779B9u + 1u};
    const uint32_t t = ctr.fetch_add(0x9E3779B9u) + 0x9E3779B9u;
    return t ? t : 0x9E3779B9u;
}

static bool fast_types(int tz, int ty, int kind) { return tz == RDK_BF16 && ty == RDK_BF16 && kind == RDK_LOGITS; }

const char* stream_ineligible(const RowParams& P, int tz, int ty, int kind, int batch, const void* ws, size_t ws_bytes) {
    const size_t es = tz == RDK_F32 ? 4 : 2, ys = ty == RDK_F32 ? 4 : 2;
    if (P.N < kStreamMinN) return "N < 4096";
    if (P.qtilde) return "q~ is written out";
    if (P.rows <= 0 || P.trials <= 0) return "no draws";
    if (P.prior) return "separate prior";
    // rows of the target start on 16-byte boundaries; drafter values are read in aligned pairs
    if ((reinterpret_cast<uintptr_t>(P.target) & 15u) || ((P.target_stride * (long long)es) & 15)) return "target rows not 16-byte aligned";
    if ((reinterpret_cast<uintptr_t>(P.drafter) & 15u) || (P.drafter_stride & 1)) return "drafter base not 16-byte aligned or odd drafter row stride";
    if ((long long)P.rows * P.trials > 0x7fffffffLL) return "too many draws";
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 15u) || ws_bytes < stream_workspace_bytes(P.rows, batch, P.trials)) return "no workspace";
    // ascending, valid kept ids only, as recorded when the index was built (the kernel re-checks the header)
    if (index_order(P.header, P.N, P.n) != 1) return "kept ids not ascending and valid (or index not prepared at this address)";
    StreamGeo g;
    if (!plan_stream(P.N, P.n, es, ys, fast_types(tz, ty, kind), g)) return "shapes beyond shared memory";
    return nullptr;
}

void set_stream_spin_limit(unsigned limit) { g_spin_limit.store(limit ? limit : kSpinLimitDefault); }

cudaError_t launch_stream_linear(RowParams P, int tz, int ty, int kind, int batch, void* ws, size_t ws_bytes, cudaStream_t s) {
    const size_t es = tz == RDK_F32 ? 4 : 2, ys = ty == RDK_F32 ? 4 : 2;
    if (stream_ineligible(P, tz, ty, kind, batch, ws, ws_bytes)) return cudaErrorNotSupported;
    StreamGeo g;
    if (!plan_stream(P.N, P.n, es, ys, fast_types(tz, ty, kind), g)) return cudaErrorNotSupported;
    g.G = 0;
    g.tag = next_tag();
    g.spin_limit = g_spin_limit.load();
    const KeptIndexView v = make_view(P.header, P.N, P.n);
    g.segdesc = v.segdesc[es == 2 ? 0 : 1];
    g.goff = v.goff[es == 2 ? 0 : 1];
    P.rec = static_cast<float*>(ws);
    P.counters = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + ws_off_counters(P.rows));
    P.xrec = reinterpret_cast<unsigned char*>(ws) + ws_off_xrec(P.rows, batch, P.trials);
    if (fast_types(tz, ty, kind)) {
        const int nst = fast_steps(g, g.nv);
        if (nst > 0) return launch_fast(P, g, nst, s);
    }
    if (tz == RDK_F32) return ty == RDK_F32 ? launch_kind_s<float, float>(P, kind, g, s) : launch_kind_s<float, __nv_bfloat16>(P, kind, g, s);
    return ty == RDK_F32 ? launch_kind_s<__nv_bfloat16, float>(P, kind, g, s) : launch_kind_s<__nv_bfloat16, __nv_bfloat16>(P, kind, g, s);
}

}  // namespace rdk

extern "C" int rdk_stream_geometry(int32_t N, int32_t n, int32_t target_dtype, int32_t drafter_dtype, rdk_stream_geometry_t* out) {
    using namespace rdk;
    if (!out || N < 1 || n < 1 || (target_dtype != RDK_F32 && target_dtype != RDK_BF16) ||
        (drafter_dtype != RDK_F32 && drafter_dtype != RDK_BF16)) {
        set_error("rdk_stream_geometry: bad argument");
        return RDK_ERR_INVALID_ARG;
    }
    const size_t es = target_dtype == RDK_F32 ? 4 : 2, ys = drafter_dtype == RDK_F32 ? 4 : 2;
    const bool ft = fast_types(target_dtype, drafter_dtype, RDK_LOGITS);
    StreamGeo g;
    *out = rdk_stream_geometry_t{};
    out->supported = plan_stream(N, n, es, ys, ft, g) ? 1 : 0;
    if (!out->supported) return RDK_OK;
    out->ctas_per_row = g.C; out->warps_per_cta = kSW; out->segment_tokens = g.Lw; out->stages = g.NS;
    out->live_rows = g.NB; out->cached_slots_per_warp = g.ycap;
    out->dynamic_shared_bytes = (int64_t)stream_smem(g, es, !(ft && fast_steps(g, g.nv) > 0));
    return RDK_OK;
}
