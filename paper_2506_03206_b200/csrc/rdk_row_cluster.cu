// Cluster kernel for the linear-time path (Eq. rdk-taylor + Algorithm 4 steps 4-8).
//
// One thread-block cluster of C CTAs takes one row.  CTA c keeps its slice of the target logits
// resident in shared memory (one TMA bulk copy), so the row is read from HBM exactly once; the
// C partial results are exchanged through distributed shared memory.
//
// Arithmetic, with p = softmax(z), q' = TLI(softmax(y)), x_j = p_j / N:
//   w_j = (N q'_j + theta p_j) / (N + p_j) = (q'_j + theta x_j) / (1 + x_j)
//       = (q'_j + theta x_j) (1 - x_j + x_j^2 - ...)                 (x_j <= 1/N <= 2^-12 here)
// * A token the drafter does not keep has q'_j = 0, hence w_j / S < p_j: its share of
//   alpha = sum min(p, q~) is w_j / S and its residual is p_j - w_j / S.  All such tokens enter only
//   through sum p_j and sum p_j^2 per segment, which come out of the soft-max sweep itself.
// * The n kept tokens are evaluated one by one (cached in shared memory as (p_j, w_j)).
// * S = sum_j w_j = 1 + (sum_j q'_j p_j^2 - theta sum_j p_j^2) / N^2 + O(N^-3), because
//   sum q' = 1 and sum q'_j p_j = theta cancel the first-order terms.
// The kernel is used for N >= 4096 only, where the truncated series is below fp32 resolution.
#include <cooperative_groups.h>

#include "rdk_row.cuh"

namespace cg = cooperative_groups;

namespace rdk {

constexpr int kCT = 256;             // threads per CTA
constexpr int kCW = kCT / 32;        // warps per CTA; each owns a contiguous token range = one CDF segment
constexpr int kMaxC = 8;             // portable cluster size
constexpr int kMaxSeg = kMaxC * kCW;
constexpr int kTrialBatch = kCW;     // trials handled between two cluster exchanges (one per warp)
constexpr int kMinClusterN = 4096;
constexpr unsigned kSpinLimit = 1u << 22;

struct Pub1 {    // per-CTA partials, published before the first exchange
    float m, my;
    float E1[kCW], E2[kCW], K1[kCW], K2[kCW], Zq[kCW], th[kCW], q2[kCW];
};
struct Pub2 { float Kw[kCW], ak[kCW]; };
struct Pub3 { int d[kTrialBatch]; float pd[kTrialBatch], wd[kTrialBatch]; };

struct CCtx {
    const void* zbuf; float2* cache; int cap;
    const uint32_t* mask; const int32_t* rank; const int32_t* slot;
    const void* yrow;
    int N, j0, r0;
    bool identity;
    float offg, inv_zp, yoffg, inv_zq, theta, inv_n, inv_s;
};

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
__device__ __forceinline__ float taylor_w(const CCtx& c, float p, float qp) {
    const float x = p * c.inv_n;
    return fmaf(c.theta, x, qp) * fmaf(x, x - 1.f, 1.f);
}

// p and w of the 8 tokens at local index jl (a multiple of 8) of this CTA's slice
template <typename TZ, typename TY, int KIND>
__device__ __forceinline__ void chunk_pw(const CCtx& c, int jl, float (&p)[kVec], float (&w)[kVec]) {
    float z[kVec];
    lds8<TZ>(static_cast<const TZ*>(c.zbuf), jl, z);
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        p[k] = ex2(fmaf(z[k], kLog2e, c.offg)) * c.inv_zp;
        w[k] = taylor_w(c, p[k], 0.f);
    }
    const int jg = c.j0 + jl;
    if (jg >= c.N) return;
    const uint32_t word = __ldg(c.mask + (jg >> 5));
    const int sh = jg & 31;
    const uint32_t mb = (word >> sh) & 0xffu;
    if (!mb) return;
    int r = __ldg(c.rank + (jg >> 5)) + __popc(word & ((1u << sh) - 1u));
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        if (mb & (1u << k)) {
            const int il = r - c.r0;
            if (il < c.cap) {
                const float2 v = c.cache[il];
                p[k] = v.x; w[k] = v.y;
            } else {
                const int i = c.identity ? r : __ldg(c.slot + r);
                const float y = to_float<TY>(static_cast<const TY*>(c.yrow)[i]);
                const float qp = (KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, c.yoffg)) : y) * c.inv_zq;
                w[k] = taylor_w(c, p[k], qp);
            }
            ++r;
        }
    }
}

enum { kPickW = 0, kPickR = 1, kPickP = 2 };

// Inverse-CDF pick inside the local token range [a, b) of this CTA's slice (one warp):
// the first token whose running sum of weights exceeds rem; if rounding leaves none, the last
// positive one.  Returns the local token index (or -1 if every weight is zero) and its p, w.
template <typename TZ, typename TY, int KIND, int WHAT>
__device__ __forceinline__ int pick_in_range(const CCtx& c, int a, int b, float rem, int lane, float& p_sel, float& w_sel) {
    float cum = 0.f;
    int last_cs = -1;
    for (int pass = 0; pass < 2; ++pass) {
        for (int cs = (pass == 0 ? a : last_cs); cs < b; cs += kSeg) {
            const int jl = cs + lane * kVec;
            float p[kVec], w[kVec], x[kVec];
#pragma unroll
            for (int k = 0; k < kVec; ++k) { p[k] = 0.f; w[k] = 0.f; }
            if (jl < b) chunk_pw<TZ, TY, KIND>(c, jl, p, w);
            float sum = 0.f;
#pragma unroll
            for (int k = 0; k < kVec; ++k) {
                x[k] = WHAT == kPickW ? w[k] : (WHAT == kPickR ? fmaxf(0.f, p[k] - w[k] * c.inv_s) : p[k]);
                sum += x[k];
            }
            sum = warp_sum(sum);
            if (sum > 0.f) {
                const bool take = pass == 1 || cum + sum > rem;
                if (take) {
                    const int sel = pick_in_segment(x, pass == 1 ? INFINITY : rem - cum, lane);
                    float ps = 0.f, ws = 0.f;
#pragma unroll
                    for (int k = 0; k < kVec; ++k) if (k == (sel & (kVec - 1))) { ps = p[k]; ws = w[k]; }
                    p_sel = __shfl_sync(0xffffffffu, ps, sel / kVec);
                    w_sel = __shfl_sync(0xffffffffu, ws, sel / kVec);
                    return cs + sel;
                }
                last_cs = cs;
                cum += sum;
            }
            if (pass == 1) break;
        }
        if (last_cs < 0) break;
    }
    p_sel = 0.f; w_sel = 0.f;
    return -1;
}

template <typename TZ, typename TY, int KIND>
__global__ void __launch_bounds__(kCT)
rdk_cluster_kernel(const RowParams P, const int C, const int Ls, const int cap) {
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(128) unsigned char dsm[];
    TZ* zbuf = reinterpret_cast<TZ*>(dsm);
    float2* cache = reinterpret_cast<float2*>(dsm + (((size_t)Ls * sizeof(TZ) + 127) & ~size_t(127)));

    __shared__ Pub1 pub1;
    __shared__ Pub2 pub2;
    __shared__ Pub3 pub3;
    __shared__ float segA[kMaxSeg], segP[kMaxSeg];
    __shared__ double cdfW[kMaxSeg], cdfR[kMaxSeg], cdfP[kMaxSeg];
    __shared__ float bc[16];
    __shared__ float redm[kCW], redy[kCW];
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int crank = (int)cluster.block_rank();
    const int row = blockIdx.x / C;

    {   // the kept-id index must belong to this problem (same decision in every CTA)
        const bool ok = P.header[kHdrMagic] == kIdxMagic && P.header[kHdrN] == P.N && P.header[kHdrn] == P.n;
        if (!ok) {
            if (tid == 0 && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_INVALID_ARG);
            return;
        }
    }
    const bool identity = P.header[kHdrIdentity] != 0;
    const int n_valid = P.header[kHdrValid];

    const int j0 = crank * Ls;
    const int len = max(0, min(P.N - j0, Ls));
    const TZ* zrow = static_cast<const TZ*>(P.target) + (long long)row * P.target_stride;
    const TY* yrow = static_cast<const TY*>(P.drafter) + (long long)row * P.drafter_stride;

    // ---- stage the slice: one thread issues the bulk copies, everybody pads the tail ------------
    const int len8 = len & ~(kVec - 1);
    const uint32_t bytes = (uint32_t)len8 * (uint32_t)sizeof(TZ);
    if (tid == 0) {
        fail = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (bytes) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&bar)), "r"(bytes) : "memory");
            const char* src = reinterpret_cast<const char*>(zrow + j0);
            for (uint32_t off = 0; off < bytes; off += 16384u) {
                const uint32_t sz = min(16384u, bytes - off);
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_u32(dsm + off)), "l"(src + off), "r"(sz), "r"(smem_u32(&bar)) : "memory");
            }
        }
    }
    for (int idx = len8 + tid; idx < Ls; idx += kCT) zbuf[idx] = idx < len ? zrow[j0 + idx] : neg_inf<TZ>();
    __syncthreads();

    // ---- drafter slice: raw values into the cache, running max ----------------------------------
    const int r0 = rank_at(P, j0, n_valid), r1 = rank_at(P, min(P.N, j0 + Ls), n_valid);
    const int kc = r1 - r0;
    float my_t = -INFINITY;
    for (int il = tid; il < kc; il += kCT) {
        const int i = identity ? r0 + il : __ldg(P.slot + r0 + il);
        const float y = to_float<TY>(yrow[i]);
        if (il < cap) cache[il].y = y;
        if (KIND == RDK_LOGITS) my_t = fmaxf(my_t, y);
    }

    if (bytes) {   // bounded wait for the bulk copies
        unsigned spins = 0;
        uint32_t done = 0;
        while (!done) {
            asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                         : "=r"(done) : "r"(smem_u32(&bar)), "r"(0u) : "memory");
            if (!done && ++spins > kSpinLimit) { atomicExch(&fail, 1); break; }
        }
    }

    // ---- slice maximum of z -------------------------------------------------------------------
    const int Lw = Ls / kCW;
    const int wa = warp * Lw, wb = wa + Lw;
    float mz_t = -INFINITY;
    for (int cs = wa; cs < wb; cs += kSeg) {
        const int jl = cs + lane * kVec;
        if (jl < wb) {
            float z[kVec];
            lds8<TZ>(zbuf, jl, z);
#pragma unroll
            for (int k = 0; k < kVec; ++k) mz_t = fmaxf(mz_t, z[k]);
        }
    }
    mz_t = warp_max(mz_t);
    my_t = warp_max(my_t);
    if (lane == 0) { redm[warp] = mz_t; redy[warp] = my_t; }
    __syncthreads();
    float m_c = redm[0], my_c = redy[0];
#pragma unroll
    for (int k = 1; k < kCW; ++k) { m_c = fmaxf(m_c, redm[k]); my_c = fmaxf(my_c, redy[k]); }
    if (KIND == RDK_PROBS) my_c = 0.f;

    // ---- soft-max sweep: sum e and sum e^2 over the warp's token range --------------------------
    const float zoff_c = -m_c * kLog2e, yoff_c = -my_c * kLog2e;
    float E1 = 0.f, E2 = 0.f;
    if (m_c > -INFINITY) {
        for (int cs = wa; cs < wb; cs += kSeg) {
            const int jl = cs + lane * kVec;
            if (jl < wb) {
                float z[kVec];
                lds8<TZ>(zbuf, jl, z);
#pragma unroll
                for (int k = 0; k < kVec; ++k) {
                    const float e = ex2(fmaf(z[k], kLog2e, zoff_c));
                    E1 += e;
                    E2 = fmaf(e, e, E2);
                }
            }
        }
    }
    // ---- kept tokens of the warp's range: e_z, e_y, their sums ------------------------------------
    const int rw0 = rank_at(P, min(P.N, j0 + wa), n_valid) - r0, rw1 = rank_at(P, min(P.N, j0 + wb), n_valid) - r0;
    float K1 = 0.f, K2 = 0.f, Zq = 0.f, th = 0.f, q2 = 0.f;
    for (int il = rw0 + lane; il < rw1; il += 32) {
        const int i = identity ? r0 + il : __ldg(P.slot + r0 + il);
        const int jl = __ldg(P.ids + i) - j0;
        const float ez = ex2(fmaf(to_float<TZ>(zbuf[jl]), kLog2e, zoff_c));
        const float y = il < cap ? cache[il].y : to_float<TY>(yrow[i]);
        const float ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff_c)) : y;
        K1 += ez;
        K2 = fmaf(ez, ez, K2);
        Zq += ey;
        th = fmaf(ez, ey, th);
        q2 = fmaf(ez * ez, ey, q2);
        if (il < cap) cache[il] = make_float2(ez, ey);
    }
    E1 = warp_sum(E1); E2 = warp_sum(E2); K1 = warp_sum(K1); K2 = warp_sum(K2);
    Zq = warp_sum(Zq); th = warp_sum(th); q2 = warp_sum(q2);
    if (lane == 0) {
        pub1.E1[warp] = E1; pub1.E2[warp] = E2; pub1.K1[warp] = K1; pub1.K2[warp] = K2;
        pub1.Zq[warp] = Zq; pub1.th[warp] = th; pub1.q2[warp] = q2;
    }
    if (tid == 0) { pub1.m = m_c; pub1.my = my_c; }
    cluster.sync();                                                            // exchange 1

    // ---- combine the C partials (warp 0 of every CTA, same order everywhere) ----------------------
    const int nseg = C * kCW;
    if (warp == 0) {
        float mc = -INFINITY, myc = -INFINITY;
        if (lane < C) {
            const Pub1* rp = cluster.map_shared_rank(&pub1, lane);
            mc = rp->m; myc = rp->my;
        }
        const float m = warp_max(mc), my = warp_max(myc);
        const float f_l = mc > -INFINITY ? ex2((mc - m) * kLog2e) : 0.f;
        const float g_l = myc > -INFINITY ? ex2((myc - my) * kLog2e) : 0.f;
        float e1[2], e2[2], k1[2], k2[2];
        float tZp = 0.f, tE2 = 0.f, tZq = 0.f, tTh = 0.f, tQ2 = 0.f;
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int s = lane + 32 * it;
            const bool valid = s < nseg;
            const int c = valid ? s / kCW : 0, w = s % kCW;
            const float f = __shfl_sync(0xffffffffu, f_l, c), g = __shfl_sync(0xffffffffu, g_l, c);
            e1[it] = e2[it] = k1[it] = k2[it] = 0.f;
            if (valid) {
                const Pub1* rp = cluster.map_shared_rank(&pub1, c);
                e1[it] = f * rp->E1[w]; e2[it] = f * f * rp->E2[w];
                k1[it] = f * rp->K1[w]; k2[it] = f * f * rp->K2[w];
                tZp += e1[it]; tE2 += e2[it];
                tZq += g * rp->Zq[w]; tTh += f * g * rp->th[w]; tQ2 += f * f * g * rp->q2[w];
            }
        }
        tZp = warp_sum(tZp); tE2 = warp_sum(tE2); tZq = warp_sum(tZq); tTh = warp_sum(tTh); tQ2 = warp_sum(tQ2);
        const float inv_zp = 1.f / tZp, inv_zq = 1.f / tZq, inv_n = 1.f / (float)P.N;
        const float theta = tTh * inv_zp * inv_zq;
        const float P2 = tE2 * inv_zp * inv_zp, Q2 = tQ2 * inv_zp * inv_zp * inv_zq;
        const float S = fmaf((Q2 - theta * P2) * inv_n, inv_n, 1.f);
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int s = lane + 32 * it;
            if (s < nseg) {
                const float Po = fmaxf(0.f, e1[it] - k1[it]) * inv_zp;
                const float P2o = fmaxf(0.f, e2[it] - k2[it]) * inv_zp * inv_zp;
                segP[s] = e1[it] * inv_zp;
                segA[s] = inv_n * (Po - inv_n * P2o);       // sum over not-kept tokens of p / (N + p)
            }
        }
        const float f_me = __shfl_sync(0xffffffffu, f_l, crank), g_me = __shfl_sync(0xffffffffu, g_l, crank);
        if (lane == 0) {
            bc[0] = -m * kLog2e; bc[1] = inv_zp; bc[2] = -my * kLog2e; bc[3] = inv_zq; bc[4] = theta;
            bc[5] = inv_n; bc[6] = 1.f / S; bc[7] = f_me * inv_zp; bc[8] = (KIND == RDK_LOGITS ? g_me : 1.f) * inv_zq;
            bc[9] = S;
        }
    }
    __syncthreads();
    CCtx c;
    c.zbuf = zbuf; c.cache = cache; c.cap = cap; c.mask = P.mask; c.rank = P.rank; c.slot = P.slot; c.yrow = yrow;
    c.N = P.N; c.j0 = j0; c.r0 = r0; c.identity = identity;
    c.offg = bc[0]; c.inv_zp = bc[1]; c.yoffg = bc[2]; c.inv_zq = bc[3]; c.theta = bc[4]; c.inv_n = bc[5]; c.inv_s = bc[6];
    const float fz = bc[7], fy = bc[8];

    // ---- kept tokens again: p, w, min(p, q~) ---------------------------------------------------
    float Kw = 0.f, ak = 0.f;
    for (int il = rw0 + lane; il < rw1; il += 32) {
        float ez, ey;
        if (il < cap) { const float2 v = cache[il]; ez = v.x; ey = v.y; }
        else {
            const int i = identity ? r0 + il : __ldg(P.slot + r0 + il);
            ez = ex2(fmaf(to_float<TZ>(zbuf[__ldg(P.ids + i) - j0]), kLog2e, zoff_c));
            const float y = to_float<TY>(yrow[i]);
            ey = KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, yoff_c)) : y;
        }
        const float p = ez * fz, qp = ey * fy;
        const float w = taylor_w(c, p, qp);
        Kw += w;
        ak += fminf(p, w * c.inv_s);
        if (il < cap) cache[il] = make_float2(p, w);
    }
    Kw = warp_sum(Kw); ak = warp_sum(ak);
    if (lane == 0) { pub2.Kw[warp] = Kw; pub2.ak[warp] = ak; }
    cluster.sync();                                                            // exchange 2

    // ---- per-segment totals and their prefix sums (fp64), row outputs -----------------------------
    if (warp == 0) {
        double sw[2], sr[2], sp[2];
        float alpha_l = 0.f;
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int s = lane + 32 * it;
            sw[it] = sr[it] = sp[it] = 0.0;
            if (s < nseg) {
                const Pub2* rp = cluster.map_shared_rank(&pub2, s / kCW);
                const float oov = c.theta * segA[s];
                const float w_s = oov + rp->Kw[s % kCW];
                const float a_s = oov * c.inv_s + rp->ak[s % kCW];
                sw[it] = (double)w_s;
                sr[it] = (double)fmaxf(0.f, segP[s] - a_s);
                sp[it] = (double)segP[s];
                alpha_l += a_s;
            }
        }
        // inclusive scan over segments: lanes hold s = lane (it 0) and s = lane + 32 (it 1)
        double iw[2], ir[2], ip[2];
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            iw[it] = sw[it]; ir[it] = sr[it]; ip[it] = sp[it];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double a = __shfl_up_sync(0xffffffffu, iw[it], o);
                const double b = __shfl_up_sync(0xffffffffu, ir[it], o);
                const double d = __shfl_up_sync(0xffffffffu, ip[it], o);
                if (lane >= o) { iw[it] += a; ir[it] += b; ip[it] += d; }
            }
        }
        const double t0w = __shfl_sync(0xffffffffu, iw[0], 31), t0r = __shfl_sync(0xffffffffu, ir[0], 31),
                     t0p = __shfl_sync(0xffffffffu, ip[0], 31);
        iw[1] += t0w; ir[1] += t0r; ip[1] += t0p;
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int s = lane + 32 * it;
            if (s < nseg) { cdfW[s] = iw[it]; cdfR[s] = ir[it]; cdfP[s] = ip[it]; }
        }
        alpha_l = warp_sum(alpha_l);
        if (lane == 0) bc[10] = alpha_l;
    }
    __syncthreads();
    const double S_d = cdfW[nseg - 1], R_d = cdfR[nseg - 1], Pt_d = cdfP[nseg - 1];
    if (crank == 0 && tid == 0) {
        if (P.alpha) P.alpha[row] = bc[10];
        if (P.theta) P.theta[row] = c.theta;
        if (P.S) P.S[row] = (float)S_d;
        if (P.residual_mass) P.residual_mass[row] = (float)R_d;
    }

    // ---- draws: one trial per warp, kTrialBatch trials between exchanges ---------------------------
    for (int t0 = 0; t0 < P.trials; t0 += kTrialBatch) {
        const int t = t0 + warp;
        const bool live = t < P.trials;
        float u0 = 0.f, u1 = 0.f, u2 = 0.f;
        int seg = 0;
        if (live) {
            const float* u = P.uniforms + ((long long)row * P.trials + t) * 4;
            u0 = __ldg(u); u1 = __ldg(u + 1); u2 = __ldg(u + 2);
            const double thr = (double)u0 * S_d;
            seg = min(first_above(cdfW, nseg, thr), nseg - 1);
            if (seg / kCW == crank) {
                const float rem = (float)(thr - (seg ? cdfW[seg - 1] : 0.0));
                const int a = (seg % kCW) * Lw;
                float pd, wd;
                int jl = pick_in_range<TZ, TY, KIND, kPickW>(c, a, a + Lw, rem, lane, pd, wd);
                if (lane == 0) { pub3.d[warp] = jl < 0 ? j0 + a : j0 + jl; pub3.pd[warp] = pd; pub3.wd[warp] = wd; }
            }
        }
        cluster.sync();                                                        // exchange 3: draft results
        if (live) {
            const Pub3* rp = cluster.map_shared_rank(&pub3, seg / kCW);
            const int d = rp->d[warp];
            const float pd = rp->pd[warp], wd = rp->wd[warp];
            const float qd = wd * c.inv_s;
            const float a_prob = (pd >= qd) ? 1.f : pd / qd;
            const bool acc = u1 * qd < pd;
            const long long o = (long long)row * P.trials + t;
            if (seg / kCW == crank && lane == 0) {
                if (P.draft_token) P.draft_token[o] = d;
                if (P.accepted) P.accepted[o] = acc ? 1 : 0;
                if (P.accept_prob) P.accept_prob[o] = a_prob;
                if (acc && P.out_token) P.out_token[o] = d;
            }
            if (!acc) {
                // residual draw from max(0, p - q~); if that has no mass, from p itself
                const bool from_p = !(R_d > 0.0);
                const double* cdf = from_p ? cdfP : cdfR;
                const double thr = (double)u2 * (from_p ? Pt_d : R_d);
                const int sr = min(first_above(cdf, nseg, thr), nseg - 1);
                if (sr / kCW == crank) {
                    const float rem = (float)(thr - (sr ? cdf[sr - 1] : 0.0));
                    const int a = (sr % kCW) * Lw;
                    float pp, ww;
                    const int jl = from_p ? pick_in_range<TZ, TY, KIND, kPickP>(c, a, a + Lw, rem, lane, pp, ww)
                                          : pick_in_range<TZ, TY, KIND, kPickR>(c, a, a + Lw, rem, lane, pp, ww);
                    if (lane == 0 && P.out_token) P.out_token[o] = jl < 0 ? j0 + a : j0 + jl;
                }
            }
        }
        cluster.sync();                                                        // all remote reads of this batch done
    }
    if (P.trials <= 0) cluster.sync();      // remote shared memory must outlive its readers
    if (tid == 0 && fail && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_TIMEOUT);
}

template <typename TZ, typename TY, int KIND>
static cudaError_t launch_one(const RowParams& P, int C, int Ls, int cap, size_t smem, cudaStream_t s) {
    auto kern = rdk_cluster_kernel<TZ, TY, KIND>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)P.rows * C, 1, 1);
    cfg.blockDim = dim3(kCT, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, P, C, Ls, cap);
}

template <typename TZ, typename TY>
static cudaError_t launch_kind_c(const RowParams& P, int kind, int C, int Ls, int cap, size_t smem, cudaStream_t s) {
    return kind == RDK_LOGITS ? launch_one<TZ, TY, RDK_LOGITS>(P, C, Ls, cap, smem, s)
                              : launch_one<TZ, TY, RDK_PROBS>(P, C, Ls, cap, smem, s);
}

cudaError_t launch_cluster_linear(const RowParams& P, int tz, int ty, int kind, cudaStream_t s) {
    const size_t es = tz == RDK_F32 ? 4 : 2;
    if (P.N < kMinClusterN || P.qtilde || P.rows <= 0) return cudaErrorNotSupported;
    if ((reinterpret_cast<uintptr_t>(P.target) & 15u) || ((P.target_stride * (long long)es) & 15)) return cudaErrorNotSupported;
    if ((long long)P.rows * kMaxC > 0x7fffffffLL) return cudaErrorNotSupported;
    // cluster size: slices of at most 32 KB where eight CTAs allow it
    int C = 1;
    while (C < kMaxC && ((size_t)P.N * es + C - 1) / C > 32768) C *= 2;
    const int per = (P.N + C - 1) / C;
    const int Ls = (per + 255) / 256 * 256;
    const long long expect = ((long long)P.n * Ls + P.N - 1) / P.N;
    long long cap = expect + expect / 8 + 64;
    const long long most = P.n < Ls ? P.n : Ls;
    if (cap > most) cap = most;
    cap = (cap + 31) / 32 * 32;
    const size_t zbytes = ((size_t)Ls * es + 127) & ~size_t(127);
    size_t smem = zbytes + (size_t)cap * sizeof(float2);
    if (smem > 200 * 1024) {
        if (zbytes > 160 * 1024) return cudaErrorNotSupported;
        cap = (long long)((200 * 1024 - zbytes) / sizeof(float2)) / 32 * 32;
        smem = zbytes + (size_t)cap * sizeof(float2);
    }
    if (tz == RDK_F32) {
        if (ty == RDK_F32) return launch_kind_c<float, float>(P, kind, C, Ls, (int)cap, smem, s);
        return launch_kind_c<float, __nv_bfloat16>(P, kind, C, Ls, (int)cap, smem, s);
    }
    if (ty == RDK_F32) return launch_kind_c<__nv_bfloat16, float>(P, kind, C, Ls, (int)cap, smem, s);
    return launch_kind_c<__nv_bfloat16, __nv_bfloat16>(P, kind, C, Ls, (int)cap, smem, s);
}

}  // namespace rdk
