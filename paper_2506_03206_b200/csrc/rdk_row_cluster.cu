// Two-kernel form of the linear-time path (Eq. rdk-taylor + Algorithm 4 steps 4-8) for N >= 4096.
//
// Kernel 1 (rdk_stream_kernel): persistent thread-block clusters of C CTAs, one row at a time.
// CTA c brings its slice of the target logits (and the matching drafter values) into shared memory
// with TMA bulk copies, so a row is read from HBM exactly once; the C partial results are exchanged
// once per row through distributed shared memory, while the next row's copies are in flight.  It leaves a
// small record per row in the workspace: the row's scalars and, for each of the C*8 contiguous
// token segments, the sums of w, of min(p, q~), of max(0, p - q~) and of p.
// Kernel 2 (rdk_draw_kernel): one CTA per (row, trial) turns the record into draws: it locates the
// segment by prefix sums over the record, re-reads that one segment (about N/64 tokens, usually
// still in L2), picks the token, runs the rejection test and the residual draw, and counts the
// accepted prefix of each sequence.
//
// Arithmetic, with p = softmax(z), q' = TLI(softmax(y)), x_j = p_j / N:
//   w_j = (N q'_j + theta p_j) / (N + p_j) = (q'_j + theta x_j) / (1 + x_j)
//       = (q'_j + theta x_j) (1 - x_j + x_j^2 - ...)                 (x_j <= 1/N <= 2^-12 here)
// * A token the drafter does not keep has q'_j = 0, hence w_j / S < p_j: its share of
//   alpha = sum min(p, q~) is w_j / S and its residual is p_j - w_j / S.  All such tokens enter only
//   through sum p_j and sum p_j^2 per segment, which come out of the soft-max sweep itself.
// * The n kept tokens are evaluated one by one from values cached in shared memory.
// * S = sum_j w_j = 1 + (sum_j q'_j p_j^2 - theta sum_j p_j^2) / N^2 + O(N^-3), because
//   sum q' = 1 and sum q'_j p_j = theta cancel the first-order terms.
#include <cooperative_groups.h>

#include "rdk_row.cuh"

namespace cg = cooperative_groups;

namespace rdk {

constexpr int kKeptPerLane = 24;     // kept tokens per lane whose ids stay in registers (768 per warp)
constexpr int kMaxCW = 16;           // warps (= segments) per CTA of kernel 1: 8 or 16
constexpr int kMaxC = 8;             // the portable cluster size (16-CTA clusters were tried: fewer resident CTAs, no gain)
constexpr int kMaxSeg = kMaxC * kMaxCW;
constexpr int kMinClusterN = 4096;
constexpr unsigned kSpinLimit = 1u << 22;
constexpr int kDT = 256;             // threads per CTA of kernel 2: 4 warps for the draft, 4 for the residual
constexpr int kGW = kDT / 64;        // warps per group of kernel 2
constexpr int kMaxChunks = 128;      // 256-token chunks per segment (N <= 2^21)

// record layout (floats): 16 scalars, then 4 per segment
enum { kRecOffg = 0, kRecInvZp, kRecYoffg, kRecInvZq, kRecTheta, kRecInvN, kRecInvS, kRecS };


struct Scal { float offg, inv_zp, yoffg, inv_zq, theta, inv_n, inv_s; };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <typename T> __device__ __forceinline__ T neg_inf();
template <> __device__ __forceinline__ float neg_inf<float>() { return -INFINITY; }
template <> __device__ __forceinline__ __nv_bfloat16 neg_inf<__nv_bfloat16>() { return __float2bfloat16_rn(-INFINITY); }

template <typename TZ> __device__ __forceinline__ void lds8(const TZ* zb, int jl, float (&v)[kVec]);
template <> __device__ __forceinline__ void lds8<__nv_bfloat16>(const __nv_bfloat16* zb, int jl, float (&v)[kVec]) {
    const uint4 q = *reinterpret_cast<const uint4*>(zb + jl);
    v[0] = bf16_lo(q.x); v[1] = bf16_hi(q.x); v[2] = bf16_lo(q.y); v[3] = bf16_hi(q.y);
    v[4] = bf16_lo(q.z); v[5] = bf16_hi(q.z); v[6] = bf16_lo(q.w); v[7] = bf16_hi(q.w);
}
template <> __device__ __forceinline__ void lds8<float>(const float* zb, int jl, float (&v)[kVec]) {
    const float4 a = *reinterpret_cast<const float4*>(zb + jl);
    const float4 b = *reinterpret_cast<const float4*>(zb + jl + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// number of kept ids below token j (j may equal N)
__device__ __forceinline__ int rank_at(const RowParams& P, int j, int n_valid) {
    if (j >= P.N) return n_valid;
    const uint32_t word = __ldg(P.mask + (j >> 5));
    return __ldg(P.rank + (j >> 5)) + __popc(word & ((1u << (j & 31)) - 1u));
}

// w_j for given p_j and q'_j:  (q' + theta x) (1 - x + x^2),  x = p / N
__device__ __forceinline__ float taylor_w(const Scal& c, float p, float qp) {
    const float x = p * c.inv_n;
    return fmaf(c.theta, x, qp) * fmaf(x, x - 1.f, 1.f);
}

__device__ __forceinline__ bool index_matches(const RowParams& P) {
    return P.header[kHdrMagic] == kIdxMagic && P.header[kHdrN] == P.N && P.header[kHdrn] == P.n;
}

// ------------------------------------------------------------------------------------------------
// kernel 1: persistent clusters.  Cluster g takes rows g, g + G, g + 2G, ...; while a row's
// partial results are exchanged and its kept tokens are revisited, the bulk copies of the next
// row's slice are already in flight.
// ------------------------------------------------------------------------------------------------
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

// running maximum over 8 consecutive logits in shared memory
template <typename TZ> struct MaxAcc;
template <> struct MaxAcc<float> {
    float m = -INFINITY;
    __device__ __forceinline__ void push(const float* zb, int jl) {
        const float4 a = *reinterpret_cast<const float4*>(zb + jl);
        const float4 b = *reinterpret_cast<const float4*>(zb + jl + 4);
        m = fmaxf(fmaxf(fmaxf(m, a.x), fmaxf(a.y, a.z)), fmaxf(fmaxf(a.w, b.x), fmaxf(b.y, fmaxf(b.z, b.w))));
    }
    __device__ __forceinline__ float result() const { return m; }
};
template <> struct MaxAcc<__nv_bfloat16> {
    __nv_bfloat162 m2 = __float2bfloat162_rn(-INFINITY);
    __device__ __forceinline__ void push(const __nv_bfloat16* zb, int jl) {
        const uint4 q = *reinterpret_cast<const uint4*>(zb + jl);
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&q.x));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&q.y));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&q.z));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&q.w));
    }
    __device__ __forceinline__ float result() const { return fmaxf(__low2float(m2), __high2float(m2)); }
};

// sum of e = 2^(z log2e + off) and of e^2 over 8 consecutive logits in shared memory (packed fp32 pairs)
template <typename TZ>
__device__ __forceinline__ void exp_sums8(const TZ* zb, int jl, float2 scale, float2 off, float2& E1, float2& E2);
template <>
__device__ __forceinline__ void exp_sums8<__nv_bfloat16>(const __nv_bfloat16* zb, int jl, float2 scale, float2 off, float2& E1, float2& E2) {
    const uint4 q = *reinterpret_cast<const uint4*>(zb + jl);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 x = ffma2(make_float2(bf16_lo(w[k]), bf16_hi(w[k])), scale, off);
        const float2 e = make_float2(ex2(x.x), ex2(x.y));
        E1 = fadd2(E1, e);
        E2 = ffma2(e, e, E2);
    }
}
template <>
__device__ __forceinline__ void exp_sums8<float>(const float* zb, int jl, float2 scale, float2 off, float2& E1, float2& E2) {
    const float4 a = *reinterpret_cast<const float4*>(zb + jl);
    const float4 b = *reinterpret_cast<const float4*>(zb + jl + 4);
    const float2 v[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y), make_float2(b.z, b.w)};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 x = ffma2(v[k], scale, off);
        const float2 e = make_float2(ex2(x.x), ex2(x.y));
        E1 = fadd2(E1, e);
        E2 = ffma2(e, e, E2);
    }
}

__device__ __forceinline__ void mbar_wait(unsigned long long* bar, uint32_t parity, int* fail) {
    unsigned spins = 0;
    uint32_t done = 0;
    while (!done) {
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (!done && ++spins > kSpinLimit) { atomicExch(fail, 1); break; }   // give up: the host reads RDK_ERR_TIMEOUT
    }
}

// One thread: arm `bar` for `bytes` and issue the bulk copies (bytes is a multiple of 16, may be 0).
__device__ __forceinline__ void bulk_load(unsigned long long* bar, void* dst, const void* src, uint32_t bytes) {
    if (bytes == 0) {
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
        return;
    }
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
    for (uint32_t off = 0; off < bytes; off += 16384u) {
        const uint32_t sz = min(16384u, bytes - off);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(static_cast<char*>(dst) + off)), "l"(static_cast<const char*>(src) + off), "r"(sz),
                       "r"(smem_u32(bar)) : "memory");
    }
}

// How the first `kcs` drafter values of a row's rank range are laid out in a y buffer: element il
// sits at index sh + il, so that the 16-byte aligned middle part can be bulk-copied.
struct YPlan { int sh, head, mid, tail; };
template <typename TY>
__device__ __forceinline__ YPlan plan_y(const TY* src, int kcs) {
    YPlan p;
    const uint32_t a = (uint32_t)(reinterpret_cast<uintptr_t>(src) & 15u);
    p.sh = (int)(a / sizeof(TY));
    p.head = min(kcs, (int)(((16u - a) & 15u) / sizeof(TY)));
    const int rest = kcs - p.head;
    p.mid = (int)(((size_t)rest * sizeof(TY) & ~size_t(15)) / sizeof(TY));
    p.tail = rest - p.mid;
    return p;
}

// address of `addr` (a shared-memory address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// 16-byte store into another CTA's shared memory that also counts 16 bytes on that CTA's mbarrier
__device__ __forceinline__ void st_async_v4(uint32_t raddr, float a, float b, float c, float d, uint32_t rbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(raddr), "f"(a), "f"(b), "f"(c), "f"(d), "r"(rbar) : "memory");
}

struct SegRec { float E1, E2, K1, K2, Zq, th, m, my; };      // one warp segment's partial sums (32 bytes)

template <typename TZ, typename TY, int KIND, int CT>
__global__ void __launch_bounds__(CT, CT == 256 ? 3 : 1)
rdk_stream_kernel(const RowParams P, const int C, const int Ls, const int cap, const int G) {
    constexpr int CW = CT / 32;          // warps per CTA; each owns a contiguous token range = one segment
    constexpr int MAXSEG = kMaxC * CW;
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(128) unsigned char dsm[];
    const size_t zb_bytes = ((size_t)Ls * sizeof(TZ) + 127) & ~size_t(127);
    const size_t yb_bytes = ((size_t)(cap + 16) * sizeof(TY) + 127) & ~size_t(127);
    TZ* zbuf = reinterpret_cast<TZ*>(dsm);
    // the two drafter buffers, addressed by arithmetic on the shared array (keeps them in the shared address space)
    auto ybuf_at = [&](int b) -> TY* { return reinterpret_cast<TY*>(dsm + zb_bytes + (b ? yb_bytes : 0)); };
    float* ezb = reinterpret_cast<float*>(dsm + zb_bytes + 2 * yb_bytes);   // e_z of the staged kept tokens

    __shared__ __align__(16) float4 segv[CW];
    __shared__ float bcs[8];
    __shared__ __align__(16) SegRec all1[2][MAXSEG];   // [row parity][segment of the row], written by the owning CTAs
    __shared__ int rk[CW + 1];
    __shared__ __align__(8) unsigned long long zbar, ybar[2], xbar[2];
    __shared__ int fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int crank = (int)cluster.block_rank();
    const int cid = blockIdx.x / C;

    if (!index_matches(P)) {   // same decision in every CTA of the grid; nothing is in flight yet
        if (tid == 0 && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_INVALID_ARG);
        return;
    }
    const bool identity = P.header[kHdrIdentity] != 0;
    const int n_valid = P.header[kHdrValid];
    // the draw kernel may be scheduled already; it waits for this whole grid before reading the records
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int j0 = crank * Ls;
    const int len = max(0, min(P.N - j0, Ls));
    const int Lw = Ls / CW;
    const int len8 = len & ~(kVec - 1);
    const uint32_t zbytes = (uint32_t)len8 * (uint32_t)sizeof(TZ);
    const int nseg = C * CW;

    if (tid == 0) {
        fail = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&zbar)));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&ybar[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&ybar[1])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&xbar[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&xbar[1])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid <= CW) rk[tid] = rank_at(P, min(P.N, j0 + tid * Lw), n_valid);   // rank at the warp range borders
    for (int idx = len + tid; idx < Ls; idx += CT) zbuf[idx] = neg_inf<TZ>();   // beyond the vocabulary: weight 0
    __syncthreads();
    cluster.sync();                       // every CTA's barriers exist before anybody signals them
    const int r0 = rk[0];
    const int kc = rk[CW] - r0;          // kept tokens of this slice
    const int kcs = min(kc, cap);         // ... of which this many are staged in shared memory

    // Loads of one row (z slice, drafter values of the slice's rank range), issued by the last warp:
    // its lanes stage the few unaligned elements with plain stores, then lane 0 arms the barriers
    // (release) and starts the bulk copies, so whoever sees a barrier complete also sees those stores.
    auto issue_loads = [&](int row, int b) {
        const TZ* zsrc = static_cast<const TZ*>(P.target) + (long long)row * P.target_stride + j0;
        const TY* ysrc = static_cast<const TY*>(P.drafter) + (long long)row * P.drafter_stride;
        if (identity) {
            if (warp == CW - 1) {
                const YPlan yp = plan_y<TY>(ysrc + r0, kcs);
                if (lane < len - len8) zbuf[len8 + lane] = zsrc[len8 + lane];
                if (lane >= 8 && lane < 8 + yp.head) { const int il = lane - 8; ybuf_at(b)[yp.sh + il] = ysrc[r0 + il]; }
                if (lane >= 16 && lane < 16 + yp.tail) { const int il = yp.head + yp.mid + lane - 16; ybuf_at(b)[yp.sh + il] = ysrc[r0 + il]; }
                __syncwarp();
                if (lane == 0) {
                    bulk_load(&zbar, zbuf, zsrc, zbytes);
                    bulk_load(&ybar[b], ybuf_at(b) + yp.sh + yp.head, ysrc + r0 + yp.head, (uint32_t)(yp.mid * sizeof(TY)));
                }
            }
        } else {
            if (tid < len - len8) zbuf[len8 + tid] = zsrc[len8 + tid];
            for (int il = tid; il < kcs; il += CT) ybuf_at(b)[il] = ysrc[__ldg(P.slot + r0 + il)];
            __syncthreads();
            if (tid == 0) { bulk_load(&zbar, zbuf, zsrc, zbytes); bulk_load(&ybar[b], nullptr, nullptr, 0); }
        }
    };
    auto y_shift = [&](int row) -> int {
        if (!identity) return 0;
        const TY* ysrc = static_cast<const TY*>(P.drafter) + (long long)row * P.drafter_stride + r0;
        return (int)((reinterpret_cast<uintptr_t>(ysrc) & 15u) / sizeof(TY));
    };

    if (cid < P.rows) issue_loads(cid, 0);
    __syncthreads();

    const int wa = warp * Lw, wb = wa + Lw;
    const int rw0 = rk[warp] - r0, rw1 = rk[warp + 1] - r0;
    const int rw1s = max(rw0, min(min(rw1, kcs), rw0 + 32 * kKeptPerLane));   // part of the warp's kept tokens handled from registers / shared memory
    // local token index of this lane's kept tokens (lane + 32 k -th of the warp's range): the same for
    // every row, so they live in registers, two 16-bit indices per word
    uint32_t idr[kKeptPerLane / 2];
#pragma unroll
    for (int k = 0; k < kKeptPerLane; ++k) {
        const int il = rw0 + lane + 32 * k;
        uint32_t v = 0;
        if (il < rw1s) v = (uint32_t)(__ldg(P.ids + (identity ? r0 + il : __ldg(P.slot + r0 + il))) - j0);
        if (k & 1) idr[k / 2] |= v << 16; else idr[k / 2] = v;
    }
    const float inv_n = 1.f / (float)P.N;
    const uint32_t xbytes = (uint32_t)nseg * (uint32_t)sizeof(SegRec);

    int it = 0;
    for (int row = cid; row < P.rows; row += G, ++it) {
        const int b = it & 1;
        const TY* yrow = static_cast<const TY*>(P.drafter) + (long long)row * P.drafter_stride;
        const TZ* zrow = static_cast<const TZ*>(P.target) + (long long)row * P.target_stride;
        const TY* yb = ybuf_at(b) + y_shift(row);
        if (tid == 0)   // this row's exchange: nseg records of 32 bytes will arrive from the cluster
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&xbar[b])), "r"(xbytes) : "memory");
        mbar_wait(&zbar, (uint32_t)(it & 1), &fail);
        mbar_wait(&ybar[b], (uint32_t)((it >> 1) & 1), &fail);

        // ---- this warp's maxima: its token range and the drafter values of its kept tokens ---------
        MaxAcc<TZ> mz;
        for (int cs = wa; cs < wb; cs += kSeg) {
            const int jl = cs + lane * kVec;
            if (jl < wb) mz.push(zbuf, jl);
        }
        float my_w = -INFINITY;
        if (KIND == RDK_LOGITS) {
#pragma unroll 4
            for (int il = rw0 + lane; il < rw1s; il += 32) my_w = fmaxf(my_w, to_float<TY>(yb[il]));
            for (int il = rw1s + lane; il < rw1; il += 32)
                my_w = fmaxf(my_w, to_float<TY>(yrow[identity ? r0 + il : __ldg(P.slot + r0 + il)]));
            my_w = warp_max(my_w);
        } else {
            my_w = 0.f;
        }
        const float m_w = warp_max(mz.result());

        // ---- soft-max sweep: sum e and sum e^2 over the warp's token range ----------------------------
        const float zoff_w = -m_w * kLog2e, yoff_w = -my_w * kLog2e;
        float E1 = 0.f, E2 = 0.f;
        if (m_w > -INFINITY) {
            float2 e1 = make_float2(0.f, 0.f), e2 = make_float2(0.f, 0.f);
            const float2 sc = make_float2(kLog2e, kLog2e), of = make_float2(zoff_w, zoff_w);
#pragma unroll 2
            for (int cs = wa; cs < wb; cs += kSeg) {
                const int jl = cs + lane * kVec;
                if (jl < wb) exp_sums8<TZ>(zbuf, jl, sc, of, e1, e2);
            }
            E1 = e1.x + e1.y; E2 = e2.x + e2.y;
        }
        // ---- kept tokens of the warp's range: e_z, e_y (cached), their sums -----------------------------
        float K1 = 0.f, K2 = 0.f, Zq = 0.f, th = 0.f;
        // groups of four per lane: all loads of a group are issued before its arithmetic and stores
#pragma unroll
        for (int g4 = 0; g4 < kKeptPerLane / 4; ++g4) {
            if (rw0 + 128 * g4 >= rw1s) break;                    // warp-uniform
            float zz[4], yy[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int k = 4 * g4 + u;
                const int il = rw0 + lane + 32 * k;
                const uint32_t jl = (k & 1) ? (idr[k / 2] >> 16) : (idr[k / 2] & 0xffffu);
                const bool ok = il < rw1s;
                zz[u] = ok ? to_float<TZ>(zbuf[jl]) : -INFINITY;
                yy[u] = ok ? to_float<TY>(yb[il]) : (KIND == RDK_LOGITS ? -INFINITY : 0.f);
            }
            float ez[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                ez[u] = ex2(fmaf(zz[u], kLog2e, zoff_w));
                const float ey = KIND == RDK_LOGITS ? ex2(fmaf(yy[u], kLog2e, yoff_w)) : yy[u];
                K1 += ez[u]; K2 = fmaf(ez[u], ez[u], K2); Zq += ey; th = fmaf(ez[u], ey, th);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int il = rw0 + lane + 32 * (4 * g4 + u);
                if (il < rw1s) ezb[il] = ez[u];
            }
        }
        for (int il = rw1s + lane; il < rw1; il += 32) {               // kept tokens beyond the staged part
            const int i = identity ? r0 + il : __ldg(P.slot + r0 + il);
            const float ez = ex2(fmaf(to_float<TZ>(zbuf[__ldg(P.ids + i) - j0]), kLog2e, zoff_w));
            const float y = to_float<TY>(yrow[i]);
            const float ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff_w)) : y;
            K1 += ez; K2 = fmaf(ez, ez, K2); Zq += ey; th = fmaf(ez, ey, th);
        }
        E1 = warp_sum(E1); E2 = warp_sum(E2); K1 = warp_sum(K1); K2 = warp_sum(K2);
        Zq = warp_sum(Zq); th = warp_sum(th);
        // push this warp's record into every CTA of the cluster (lane c writes to CTA c)
        if (lane < C) {
            const uint32_t raddr = mapa_u32(smem_u32(&all1[b][crank * CW + warp]), (uint32_t)lane);
            const uint32_t rbar = mapa_u32(smem_u32(&xbar[b]), (uint32_t)lane);
            st_async_v4(raddr, E1, E2, K1, K2, rbar);
            st_async_v4(raddr + 16, Zq, th, m_w, my_w, rbar);
        }
        __syncthreads();                  // every warp is done with zbuf: the next row may stream in
        if (row + G < P.rows) issue_loads(row + G, b ^ 1);
        mbar_wait(&xbar[b], (uint32_t)((it >> 1) & 1), &fail);                 // all nseg records have arrived

        // ---- combine the records (warp 0), hand every warp its scalars through shared memory --------
        if (warp == 0) {
            float e1[MAXSEG / 32], e2[MAXSEG / 32], k1[MAXSEG / 32], k2[MAXSEG / 32], zq[MAXSEG / 32], tt[MAXSEG / 32];
            float ms[MAXSEG / 32], mys[MAXSEG / 32];
            float m = -INFINITY, my = -INFINITY;
#pragma unroll
            for (int q = 0; q < MAXSEG / 32; ++q) {
                const int s = lane + 32 * q;
                e1[q] = e2[q] = k1[q] = k2[q] = zq[q] = tt[q] = 0.f; ms[q] = mys[q] = -INFINITY;
                if (s < nseg) {
                    const float4 u = *reinterpret_cast<const float4*>(&all1[b][s]);
                    const float4 v = *(reinterpret_cast<const float4*>(&all1[b][s]) + 1);
                    e1[q] = u.x; e2[q] = u.y; k1[q] = u.z; k2[q] = u.w; zq[q] = v.x; tt[q] = v.y; ms[q] = v.z; mys[q] = v.w;
                }
                m = fmaxf(m, ms[q]); my = fmaxf(my, mys[q]);
            }
            m = warp_max(m); my = warp_max(my);
            float tZp = 0.f, tZq = 0.f, tTh = 0.f, f_q[MAXSEG / 32], g_q[MAXSEG / 32];
#pragma unroll
            for (int q = 0; q < MAXSEG / 32; ++q) {
                const float f = ms[q] > -INFINITY ? ex2((ms[q] - m) * kLog2e) : 0.f;
                const float g = mys[q] > -INFINITY ? ex2((mys[q] - my) * kLog2e) : 0.f;
                f_q[q] = f; g_q[q] = g;
                e1[q] *= f; e2[q] *= f * f; k1[q] *= f; k2[q] *= f * f;
                tZp += e1[q]; tZq += g * zq[q]; tTh += f * g * tt[q];
            }
            tZp = warp_sum(tZp); tZq = warp_sum(tZq); tTh = warp_sum(tTh);
            const float inv_zp = 1.f / tZp, inv_zq = 1.f / tZq;
            const float theta = tTh * inv_zp * inv_zq;
            // own segments: total p mass, sum over the not-kept tokens of p / (N + p), scales
#pragma unroll
            for (int q = 0; q < MAXSEG / 32; ++q) {
                const int s = lane + 32 * q;
                if (s < nseg && s / CW == crank) {
                    const float Po = fmaxf(0.f, e1[q] - k1[q]) * inv_zp;
                    const float P2o = fmaxf(0.f, e2[q] - k2[q]) * inv_zp * inv_zp;
                    segv[s % CW] = make_float4(e1[q] * inv_zp, inv_n * (Po - inv_n * P2o), f_q[q] * inv_zp,
                                                (KIND == RDK_LOGITS ? g_q[q] : 1.f) * inv_zq);
                }
            }
            if (lane == 0) { bcs[0] = -m * kLog2e; bcs[1] = inv_zp; bcs[2] = -my * kLog2e; bcs[3] = inv_zq; bcs[4] = theta; }
        }
        __syncthreads();
        Scal c;
        c.offg = bcs[0]; c.inv_zp = bcs[1]; c.yoffg = bcs[2]; c.inv_zq = bcs[3]; c.theta = bcs[4];
        c.inv_n = inv_n; c.inv_s = 1.f;      // S = 1 - theta sum p^2 / N^2 + ... rounds to 1 in fp32 for N >= 4096 (|S - 1| < 2^-24)
        const float S_row = 1.f;
        const float4 sv = segv[warp];
        const float segP_w = sv.x, segA_w = sv.y, fz = sv.z, fy = sv.w;

        // ---- kept tokens again: sum of min(p, q~) --------------------------------------------------
        float ak = 0.f;
#pragma unroll 4
        for (int il = rw0 + lane; il < rw1s; il += 32) {
            const float y = to_float<TY>(yb[il]);
            const float ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff_w)) : y;
            const float p = ezb[il] * fz;
            ak += fminf(p, taylor_w(c, p, ey * fy) * c.inv_s);
        }
        for (int il = rw1s + lane; il < rw1; il += 32) {
            const int i = identity ? r0 + il : __ldg(P.slot + r0 + il);
            const float ez = ex2(fmaf(to_float<TZ>(zrow[__ldg(P.ids + i)]), kLog2e, zoff_w));
            const float y = to_float<TY>(yrow[i]);
            const float ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff_w)) : y;
            const float p = ez * fz;
            ak += fminf(p, taylor_w(c, p, ey * fy) * c.inv_s);
        }
        ak = warp_sum(ak);

        // ---- the row's record -------------------------------------------------------------------------
        float* rec = P.rec + (long long)row * kRecFloats;
        if (lane == 0) {
            // sum over the segment's kept tokens of w = (q' + theta x)(1 - x + x^2), x = p / N, from the
            // moments of pass 1 (terms of relative size x^2 <= 2^-24 dropped)
            const float xs = fz * c.inv_n;
            const float Kw = fy * Zq - fy * xs * th + c.theta * (xs * K1 - xs * xs * K2);
            const float oov = c.theta * segA_w;
            const float a_s = oov * c.inv_s + ak;
            reinterpret_cast<float4*>(rec + 16)[crank * CW + warp] = make_float4(oov + Kw, a_s, fmaxf(0.f, segP_w - a_s), segP_w);
        }
        if (crank == 0) {
            if (tid == 0) {
                rec[kRecOffg] = c.offg; rec[kRecInvZp] = c.inv_zp; rec[kRecYoffg] = c.yoffg; rec[kRecInvZq] = c.inv_zq;
                rec[kRecTheta] = c.theta; rec[kRecInvN] = c.inv_n; rec[kRecInvS] = c.inv_s; rec[kRecS] = S_row;
            }
            if (P.counters && row % P.positions == 0)
                for (int t = tid; t < P.trials; t += CT) P.counters[(row / P.positions) * P.trials + t] = 0;
        }
    }
    if (tid == 0 && fail && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_TIMEOUT);
    cluster.sync();                        // no CTA leaves while others may still write into it
}

// ------------------------------------------------------------------------------------------------
// kernel 2
// ------------------------------------------------------------------------------------------------
struct DrawCtx {
    const void* zrow; const void* yrow; bool zvec;
    const uint32_t* mask; const int32_t* rank; const int32_t* slot;
    int N; bool identity;
    Scal c;
};

// p and w of the 8 tokens starting at global token jb (a multiple of 8)
template <typename TZ, typename TY, int KIND>
__device__ __forceinline__ void draw_pw(const DrawCtx& d, int jb, float (&p)[kVec], float (&w)[kVec]) {
    float z[kVec];
    load8<TZ>(static_cast<const TZ*>(d.zrow), jb, d.N, d.zvec, -INFINITY, z);
    const uint32_t word = __ldg(d.mask + (jb >> 5));
    const int rbase = __ldg(d.rank + (jb >> 5));          // issued together with the mask and the logits
    const int sh = jb & 31;
    const uint32_t mb = (word >> sh) & 0xffu;
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        p[k] = ex2(fmaf(z[k], kLog2e, d.c.offg)) * d.c.inv_zp;
        w[k] = taylor_w(d.c, p[k], 0.f);
    }
    if (!mb) return;
    int r = rbase + __popc(word & ((1u << sh) - 1u));
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        if (mb & (1u << k)) {
            const int i = d.identity ? r : __ldg(d.slot + r);
            ++r;
            const float y = to_float<TY>(static_cast<const TY*>(d.yrow)[i]);
            const float qp = (KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, d.c.yoffg)) : y) * d.c.inv_zq;
            w[k] = taylor_w(d.c, p[k], qp);
        }
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

template <typename TZ, typename TY, int KIND>
__global__ void __launch_bounds__(kDT)
rdk_draw_kernel(const RowParams P, const int C, const int Ls, const int cw) {
    __shared__ double cdfW[kMaxSeg], cdfR[kMaxSeg], cdfP[kMaxSeg];
    __shared__ float sums[2][kMaxChunks];
    __shared__ float alpha_s;
    __shared__ int res_tok[2];
    __shared__ float res_p[2], res_w[2];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x / P.trials, t = blockIdx.x % P.trials;
    const float* rec = P.rec + (long long)row * kRecFloats;
    const int nseg = C * cw, Lw = Ls / cw;
    DrawCtx d;
    const float* u = P.uniforms + ((long long)row * P.trials + t) * 4;
    const float u0 = __ldg(u), u1 = __ldg(u + 1), u2 = __ldg(u + 2);
    d.identity = P.header[kHdrIdentity] != 0;
    if (!index_matches(P)) return;                 // kernel 1 has reported it
    asm volatile("griddepcontrol.wait;" ::: "memory");   // kernel 1 (launched just before) is complete and visible
    d.c.offg = __ldcg(rec + kRecOffg); d.c.inv_zp = __ldcg(rec + kRecInvZp); d.c.yoffg = __ldcg(rec + kRecYoffg);
    d.c.inv_zq = __ldcg(rec + kRecInvZq); d.c.theta = __ldcg(rec + kRecTheta); d.c.inv_n = __ldcg(rec + kRecInvN);
    d.c.inv_s = __ldcg(rec + kRecInvS);

    if (warp == 0) {   // prefix sums over the segments, fp64
        constexpr int Q = kMaxSeg / 32;
        double iw[Q], ir[Q], ip[Q];
        double cw = 0.0, cr = 0.0, cp = 0.0;
        float alpha_l = 0.f;
#pragma unroll
        for (int it = 0; it < Q; ++it) {
            const int s = lane + 32 * it;
            iw[it] = ir[it] = ip[it] = 0.0;
            if (s < nseg) {
                const float4 v = __ldcg(reinterpret_cast<const float4*>(rec + 16) + s);
                iw[it] = (double)v.x; alpha_l += v.y; ir[it] = (double)v.z; ip[it] = (double)v.w;
            }
        }
#pragma unroll
        for (int it = 0; it < Q; ++it) {
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double a = __shfl_up_sync(0xffffffffu, iw[it], o);
                const double b = __shfl_up_sync(0xffffffffu, ir[it], o);
                const double e = __shfl_up_sync(0xffffffffu, ip[it], o);
                if (lane >= o) { iw[it] += a; ir[it] += b; ip[it] += e; }
            }
            iw[it] += cw; ir[it] += cr; ip[it] += cp;
            cw = __shfl_sync(0xffffffffu, iw[it], 31);
            cr = __shfl_sync(0xffffffffu, ir[it], 31);
            cp = __shfl_sync(0xffffffffu, ip[it], 31);
            const int s = lane + 32 * it;
            if (s < nseg) { cdfW[s] = iw[it]; cdfR[s] = ir[it]; cdfP[s] = ip[it]; }
        }
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
    d.mask = P.mask; d.rank = P.rank; d.slot = P.slot; d.N = P.N;

    // group 0 (first half of the warps): the draft draw from w; group 1: the residual draw, computed
    // alongside (it is only used if the draft is rejected)
    const int g = warp / kGW, wg = warp % kGW;
    const bool from_p = !(R_d > 0.0);                 // p and q~ coincide: the replacement comes from p itself
    const double* cdf = g == 0 ? cdfW : (from_p ? cdfP : cdfR);
    const int what = g == 0 ? kPickW : (from_p ? kPickP : kPickR);
    const double thr = g == 0 ? (double)u0 * S_d : (double)u2 * (from_p ? Pt_d : R_d);
    const int seg = min(first_above(cdf, nseg, thr), nseg - 1);
    const float rem = (float)(thr - (seg ? cdf[seg - 1] : 0.0));
    const int seg_lo = (seg / cw) * Ls + (seg % cw) * Lw;
    const int seg_end = min(P.N, seg_lo + Lw);
    const int nch = (Lw + kSeg - 1) / kSeg;
    for (int ch = wg; ch < nch; ch += kGW) {
        float p[kVec], w[kVec], x[kVec];
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
            float p[kVec], w[kVec], x[kVec];
            draw_x<TZ, TY, KIND>(d, what, seg_lo + chosen * kSeg + lane * kVec, seg_end, p, w, x);
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
struct Geometry { int C, Ls, cap, ct; size_t smem; };

static bool plan_geometry(int N, int n, size_t es, size_t ys, int max_c, int ct, Geometry& g) {
    const int kCW = ct / 32;
    int C = 1;
    while (C < max_c && ((size_t)N * es + C - 1) / C > 32768) C *= 2;      // slices of at most 32 KB if 8 CTAs allow
    const int per = (N + C - 1) / C;
    const int Ls = (per + 32 * kCW - 1) / (32 * kCW) * (32 * kCW);
    const long long expect = ((long long)n * Ls + N - 1) / N;
    long long cap = expect + expect / 8 + 64;
    const long long most = n < Ls ? n : Ls;
    if (cap > most) cap = most;
    cap = (cap + 31) / 32 * 32;
    const size_t zbytes = ((size_t)Ls * es + 127) & ~size_t(127);
    auto total = [&](long long k) {
        const size_t yb = ((size_t)(k + 16) * ys + 127) & ~size_t(127);
        return zbytes + 2 * yb + (size_t)k * 4;
    };
    size_t smem = total(cap);
    if (smem > 200 * 1024) {
        if (zbytes > 160 * 1024) return false;
        cap = (long long)((200 * 1024 - zbytes - 512) / (4 + 2 * ys)) / 32 * 32;
        smem = total(cap);
    }
    if ((Ls / kCW + kSeg - 1) / kSeg > kMaxChunks || Ls > 65536) return false;   // local token indices are 16-bit
    g.C = C; g.Ls = Ls; g.cap = (int)cap; g.smem = smem; g.ct = ct;
    return true;
}

template <typename TZ, typename TY, int KIND, int CT>
static cudaError_t launch_ct(const RowParams& P, const Geometry& g, cudaStream_t s) {
    constexpr int kCT = CT;
    auto kern = rdk_stream_kernel<TZ, TY, KIND, CT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem);
    if (e != cudaSuccess) return e;
    if (g.C > 8) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)g.C, 1, 1);
    cfg.blockDim = dim3(kCT, 1, 1);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = g.C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // how many clusters fit on the device at once (cached per kernel instance, shape and device)
    static thread_local int c_dev = -1, c_C = 0, c_G = 0;
    static thread_local size_t c_smem = 0;
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev != c_dev || g.C != c_C || g.smem != c_smem) {
        int sms = 0, per_sm = 0, ncl = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kCT, g.smem);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3((unsigned)(sms * per_sm / g.C * g.C), 1, 1);
        e = cudaOccupancyMaxActiveClusters(&ncl, kern, &cfg);
        if (e != cudaSuccess) return e;
        if (ncl < 1) return cudaErrorNotSupported;
        c_dev = dev; c_C = g.C; c_smem = g.smem; c_G = ncl;
    }
    const int G = P.rows < c_G ? P.rows : c_G;
    cfg.gridDim = dim3((unsigned)G * g.C, 1, 1);
    e = cudaLaunchKernelEx(&cfg, kern, P, g.C, g.Ls, g.cap, G);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t dcfg = {};
    dcfg.gridDim = dim3((unsigned)(P.rows * P.trials), 1, 1);
    dcfg.blockDim = dim3(kDT, 1, 1);
    dcfg.dynamicSmemBytes = 0;
    dcfg.stream = s;
    cudaLaunchAttribute dattr[1];
    dattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while kernel 1 drains
    dattr[0].val.programmaticStreamSerializationAllowed = 1;
    dcfg.attrs = dattr;
    dcfg.numAttrs = 1;
    return cudaLaunchKernelEx(&dcfg, rdk_draw_kernel<TZ, TY, KIND>, P, g.C, g.Ls, CT / 32);
}

template <typename TZ, typename TY, int KIND>
static cudaError_t launch_one(const RowParams& P, const Geometry& g, cudaStream_t s) {
    return g.ct == 256 ? launch_ct<TZ, TY, KIND, 256>(P, g, s) : launch_ct<TZ, TY, KIND, 512>(P, g, s);
}

template <typename TZ, typename TY>
static cudaError_t launch_kind_c(const RowParams& P, int kind, const Geometry& g, cudaStream_t s) {
    return kind == RDK_LOGITS ? launch_one<TZ, TY, RDK_LOGITS>(P, g, s) : launch_one<TZ, TY, RDK_PROBS>(P, g, s);
}

size_t cluster_workspace_bytes(int rows, int batch, int trials) {
    return idx_align((size_t)rows * kRecFloats * sizeof(float)) + idx_align((size_t)batch * trials * sizeof(int32_t));
}

cudaError_t launch_cluster_linear(RowParams P, int tz, int ty, int kind, int batch, void* ws, size_t ws_bytes, cudaStream_t s) {
    const size_t es = tz == RDK_F32 ? 4 : 2;
    if (P.N < kMinClusterN || P.qtilde || P.rows <= 0 || P.trials <= 0 || !ws) return cudaErrorNotSupported;
    if ((reinterpret_cast<uintptr_t>(P.target) & 15u) || ((P.target_stride * (long long)es) & 15)) return cudaErrorNotSupported;
    if ((long long)P.rows * kMaxC > 0x7fffffffLL || (long long)P.rows * P.trials > 0x7fffffffLL) return cudaErrorNotSupported;
    if ((reinterpret_cast<uintptr_t>(ws) & 15u) || ws_bytes < cluster_workspace_bytes(P.rows, batch, P.trials)) return cudaErrorNotSupported;
    P.rec = static_cast<float*>(ws);
    P.counters = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + idx_align((size_t)P.rows * kRecFloats * sizeof(float)));
    cudaError_t e = cudaErrorNotSupported;
    for (int max_c = kMaxC; max_c >= 8 && e == cudaErrorNotSupported; max_c /= 2) {   // 16-CTA clusters first, then 8
        Geometry g;
        if (!plan_geometry(P.N, P.n, es, ty == RDK_F32 ? 4 : 2, max_c, 256, g)) continue;
        // a slice so large that only one CTA fits per SM gets 16 warps instead of 8
        if (g.smem > 110 * 1024 && !plan_geometry(P.N, P.n, es, ty == RDK_F32 ? 4 : 2, max_c, 512, g)) continue;
        if (tz == RDK_F32) e = ty == RDK_F32 ? launch_kind_c<float, float>(P, kind, g, s) : launch_kind_c<float, __nv_bfloat16>(P, kind, g, s);
        else e = ty == RDK_F32 ? launch_kind_c<__nv_bfloat16, float>(P, kind, g, s) : launch_kind_c<__nv_bfloat16, __nv_bfloat16>(P, kind, g, s);
        if (g.C <= 8) break;
        if (e != cudaSuccess && e != cudaErrorNotSupported) { (void)cudaGetLastError(); e = cudaErrorNotSupported; }   // 16 not schedulable here
    }
    return e;
}

}  // namespace rdk
