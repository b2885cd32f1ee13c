// Row kernel: one CTA takes one row (sequence, draft position) through
//   soft-max statistics of the target and drafter logits            (Sec. 4.1 soft-max)
//   Token-Level Intersection                                        (Eq. tli-drafter)
//   first-order redistribution  theta = p^T q',
//        w_j = (N q'_j + theta p_j) / (N + p_j),  S = sum_j w_j      (Eq. rdk-taylor)
//     or a pre-computed w = M^T q' read from memory                  (Algorithm 1 step 2)
//   draft draw d ~ w / S, test min(1, p_d / q~_d), acceptance rate alpha = sum min(p, q~)
//   (Definition 2.1) and the residual draw from max(0, p - q~)       (Algorithm 4 steps 4-8).
// Nothing N-long is written unless the caller asks for q~ itself.
#include <stdlib.h>

#include "rdk_row.cuh"

namespace rdk {

struct RowCtx {
    int N, tid, lane, warp;
    bool zvec, wvec, identity;
    float zoff, inv_zp, yoff, inv_zq, theta, Nf, inv_s;
    float poff, inv_zpi;      // soft-max of the prior, when there is one
    bool pvec;
};

// p and w of the kVec tokens starting at `base` (tokens at or beyond N give p = w = 0).
template <typename TZ, typename TY, int MODE, int KIND>
__device__ __forceinline__ void load_pw(const RowParams& P, const RowCtx& c, const TZ* __restrict__ zrow,
                                        const TY* __restrict__ yrow, const float* __restrict__ wrow,
                                        int base, float (&p)[kVec], float (&w)[kVec]) {
    float z[kVec];
    load8<TZ>(zrow, base, c.N, c.zvec, -INFINITY, z);
#pragma unroll
    for (int k = 0; k < kVec; ++k) p[k] = ex2(fmaf(z[k], kLog2e, c.zoff)) * c.inv_zp;
    if (MODE == RDK_MODE_PRECOMPUTED_W) {
        load8<float>(wrow, base, c.N, c.wvec, 0.f, w);
        return;
    }
    float qp[kVec];
#pragma unroll
    for (int k = 0; k < kVec; ++k) qp[k] = 0.f;
    const uint32_t word = __ldg(P.mask + (base >> 5));
    const int sh = base & 31;
    const uint32_t mb = (word >> sh) & 0xffu;
    if (mb) {
        int r = __ldg(P.rank + (base >> 5)) + __popc(word & ((1u << sh) - 1u));
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
            if (mb & (1u << k)) {
                const int i = c.identity ? r : __ldg(P.slot + r);
                ++r;
                const float y = to_float<TY>(yrow[i]);
                qp[k] = (KIND == RDK_LOGITS ? ex2(fmaf(y, kLog2e, c.yoff)) : y) * c.inv_zq;
            }
        }
    }
#pragma unroll
    if (P.prior) {    // Eq. rdk-taylor with the prior's distribution pi in place of p
        const TZ* prow = static_cast<const TZ*>(P.prior) + (long long)blockIdx.x * P.prior_stride;
        float pr[kVec];
        load8<TZ>(prow, base, c.N, c.pvec, -INFINITY, pr);
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
            const float pi = ex2(fmaf(pr[k], kLog2e, c.poff)) * c.inv_zpi;
            w[k] = (c.Nf * qp[k] + c.theta * pi) / (c.Nf + pi);
        }
        return;
    }
#pragma unroll
    for (int k = 0; k < kVec; ++k) w[k] = (c.Nf * qp[k] + c.theta * p[k]) / (c.Nf + p[k]);
}

template <typename TZ, typename TY, int MODE, int KIND>
__global__ void __launch_bounds__(kRowThreads)
rdk_row_kernel(const RowParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int num_segs = P.num_tiles * kRowWarps;
    double* cdf_w = reinterpret_cast<double*>(smem_raw);
    double* cdf_r = cdf_w + num_segs;
    float* seg_w = reinterpret_cast<float*>(cdf_r + num_segs);
    float* seg_r = seg_w + num_segs;

    __shared__ MS red_z[kRowWarps], red_y[kRowWarps], red_t[kRowWarps], red_p[kRowWarps];
    __shared__ float red_q[kRowWarps];
    __shared__ double red_a[kRowWarps];
    __shared__ float bc[8];
    __shared__ double bc_d[2];

    const int row = blockIdx.x;
    RowCtx c;
    c.N = P.N; c.tid = threadIdx.x; c.lane = threadIdx.x & 31; c.warp = threadIdx.x >> 5;
    c.Nf = (float)P.N;
    c.identity = true;

    if (MODE == RDK_MODE_LINEAR) {
        const bool ok = P.header[kHdrMagic] == kIdxMagic && P.header[kHdrN] == P.N && P.header[kHdrn] == P.n;
        if (!ok) {   // the kept-id index does not belong to this problem: refuse, uniformly
            if (threadIdx.x == 0 && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_INVALID_ARG);
            return;
        }
        c.identity = P.header[kHdrIdentity] != 0;
    }

    const TZ* zrow = static_cast<const TZ*>(P.target) + (long long)row * P.target_stride;
    const TY* yrow = (MODE == RDK_MODE_LINEAR) ? static_cast<const TY*>(P.drafter) + (long long)row * P.drafter_stride : nullptr;
    const float* wrow = (MODE == RDK_MODE_PRECOMPUTED_W) ? P.w + (long long)row * P.w_stride : nullptr;
    c.zvec = (reinterpret_cast<uintptr_t>(zrow) & 15u) == 0;
    c.wvec = wrow && (reinterpret_cast<uintptr_t>(wrow) & 15u) == 0;
    const bool has_prior = MODE == RDK_MODE_LINEAR && P.prior != nullptr;
    const TZ* prow = has_prior ? static_cast<const TZ*>(P.prior) + (long long)row * P.prior_stride : nullptr;
    c.pvec = prow && (reinterpret_cast<uintptr_t>(prow) & 15u) == 0;
    c.poff = 0.f; c.inv_zpi = 1.f;

    // ---- pass 1: soft-max statistics (running max / sum), theta numerator ----------------------
    MS zs{-INFINITY, 0.f, 0.f}, ys{-INFINITY, 0.f, 0.f}, ts{-INFINITY, 0.f, 0.f}, ps{-INFINITY, 0.f, 0.f};
    float sq = 0.f;
    for (int tile = 0; tile < P.num_tiles; ++tile) {
        const int base = tile * kTile + c.tid * kVec;
        if (MODE == RDK_MODE_LINEAR && base >= P.N) break;
        float wsum_t = 0.f;
        if (base < P.N) {
            if (MODE == RDK_MODE_PRECOMPUTED_W) {       // w does not depend on the soft-max: its sums ride along
                float w8[kVec];
                load8<float>(wrow, base, P.N, c.wvec, 0.f, w8);
#pragma unroll
                for (int k = 0; k < kVec; ++k) wsum_t += w8[k];
            }
            float z[kVec], e[kVec];
            load8<TZ>(zrow, base, P.N, c.zvec, -INFINITY, z);
            float vmax = z[0];
#pragma unroll
            for (int k = 1; k < kVec; ++k) vmax = fmaxf(vmax, z[k]);
            if (vmax > -INFINITY || MODE == RDK_MODE_LINEAR) {   // (kept drafter values count even where every target logit is -inf)
                if (vmax > zs.m) {
                    const float sc = ex2((zs.m - vmax) * kLog2e);
                    zs.s *= sc; zs.b *= sc; zs.m = vmax;
                }
                const float off = zs.m > -INFINITY ? -zs.m * kLog2e : 0.f;
#pragma unroll
                for (int k = 0; k < kVec; ++k) { e[k] = ex2(fmaf(z[k], kLog2e, off)); zs.s += e[k]; }
                float pr[kVec], ep[kVec];
                if (has_prior) {      // the prior's soft-max statistics; theta is then taken with the prior
                    load8<TZ>(prow, base, P.N, c.pvec, -INFINITY, pr);
                    float pmax = pr[0];
#pragma unroll
                    for (int k = 1; k < kVec; ++k) pmax = fmaxf(pmax, pr[k]);
                    if (pmax > ps.m) {
                        const float sc = ex2((ps.m - pmax) * kLog2e);
                        ps.s *= sc; ps.b *= sc; ps.m = pmax;
                    }
                    const float poff = ps.m > -INFINITY ? -ps.m * kLog2e : 0.f;
#pragma unroll
                    for (int k = 0; k < kVec; ++k) { ep[k] = ex2(fmaf(pr[k], kLog2e, poff)); ps.s += ep[k]; }
                }
                if (MODE == RDK_MODE_LINEAR) {
                    const uint32_t word = __ldg(P.mask + (base >> 5));
                    const int sh = base & 31;
                    const uint32_t mb = (word >> sh) & 0xffu;
                    if (mb) {
                        int r = __ldg(P.rank + (base >> 5)) + __popc(word & ((1u << sh) - 1u));
#pragma unroll
                        for (int k = 0; k < kVec; ++k) {
                            if (mb & (1u << k)) {
                                const int i = c.identity ? r : __ldg(P.slot + r);
                                ++r;
                                const float y = to_float<TY>(yrow[i]);
                                if (KIND == RDK_LOGITS) { ms_push(ys, y); ms_push(ts, (has_prior ? pr[k] : z[k]) + y); }
                                else { sq += y; if (has_prior) ps.b += ep[k] * y; else zs.b += e[k] * y; }
                            }
                        }
                    }
                }
            }
        }
        if (MODE == RDK_MODE_PRECOMPUTED_W) {
            wsum_t = warp_sum(wsum_t);
            if (c.lane == 0) seg_w[tile * kRowWarps + c.warp] = wsum_t;
        }
    }
    zs = ms_warp(zs);
    if (has_prior) ps = ms_warp(ps);
    if (MODE == RDK_MODE_LINEAR) {
        if (KIND == RDK_LOGITS) { ys = ms_warp(ys); ts = ms_warp(ts); }
        else sq = warp_sum(sq);
    }
    if (c.lane == 0) { red_z[c.warp] = zs; red_y[c.warp] = ys; red_t[c.warp] = ts; red_q[c.warp] = sq; red_p[c.warp] = ps; }
    __syncthreads();
    if (c.warp == 0) {
        MS a = (c.lane < kRowWarps) ? red_z[c.lane] : MS{-INFINITY, 0.f, 0.f};
        MS b = (c.lane < kRowWarps) ? red_y[c.lane] : MS{-INFINITY, 0.f, 0.f};
        MS t = (c.lane < kRowWarps) ? red_t[c.lane] : MS{-INFINITY, 0.f, 0.f};
        float q = (c.lane < kRowWarps) ? red_q[c.lane] : 0.f;
        MS pa = (has_prior && c.lane < kRowWarps) ? red_p[c.lane] : MS{-INFINITY, 0.f, 0.f};
        a = ms_warp(a); b = ms_warp(b); t = ms_warp(t); q = warp_sum(q);
        if (has_prior) pa = ms_warp(pa);
        if (c.lane == 0) {
            float theta = 0.f, zq = 1.f, my = 0.f;
            const MS pi = has_prior ? pa : a;            // the distribution that enters theta
            if (MODE == RDK_MODE_LINEAR) {
                if (KIND == RDK_LOGITS) {
                    zq = b.s; my = b.m;
                    theta = (t.m == -INFINITY) ? 0.f : t.s * ex2((t.m - pi.m - b.m) * kLog2e) / (pi.s * b.s);
                } else {
                    zq = q;
                    theta = pi.b / (pi.s * q);
                }
            }
            bc[0] = a.m; bc[1] = a.s; bc[2] = my; bc[3] = zq; bc[4] = theta; bc[6] = pi.m; bc[7] = pi.s;
        }
    }
    __syncthreads();
    c.zoff = -bc[0] * kLog2e;
    c.inv_zp = 1.f / bc[1];
    c.yoff = -bc[2] * kLog2e;
    c.inv_zq = 1.f / bc[3];
    c.theta = bc[4];
    c.poff = -bc[6] * kLog2e;
    c.inv_zpi = 1.f / bc[7];

    // ---- pass 2: S = sum_j w_j and the per-segment sums of w (done in pass 1 for a given w) -------
    for (int tile = 0; MODE == RDK_MODE_LINEAR && tile < P.num_tiles; ++tile) {
        const int base = tile * kTile + c.tid * kVec;
        float sum = 0.f;
        if (base < P.N) {
            float p[kVec], w[kVec];
            load_pw<TZ, TY, MODE, KIND>(P, c, zrow, yrow, wrow, base, p, w);
#pragma unroll
            for (int k = 0; k < kVec; ++k) sum += w[k];
        }
        sum = warp_sum(sum);
        if (c.lane == 0) seg_w[tile * kRowWarps + c.warp] = sum;
    }
    __syncthreads();
    if (c.warp == 0) {
        const double tot = warp_scan_segments(seg_w, cdf_w, num_segs, c.lane);
        if (c.lane == 0) bc_d[0] = tot;
    }
    __syncthreads();
    const double S_d = bc_d[0];
    const float S = (float)S_d;
    c.inv_s = (MODE == RDK_MODE_PRECOMPUTED_W && P.w_as_given) ? 1.f : 1.f / S;

    // ---- pass 3: alpha = sum min(p, q~), residual sums, optional q~ output ----------------------
    float* qrow = P.qtilde ? P.qtilde + (long long)row * P.N : nullptr;
    const bool qvec = qrow && (reinterpret_cast<uintptr_t>(qrow) & 15u) == 0;
    float alpha_loc = 0.f;
    for (int tile = 0; tile < P.num_tiles; ++tile) {
        const int base = tile * kTile + c.tid * kVec;
        float rsum = 0.f;
        if (base < P.N) {
            float p[kVec], w[kVec], qt[kVec];
            load_pw<TZ, TY, MODE, KIND>(P, c, zrow, yrow, wrow, base, p, w);
#pragma unroll
            for (int k = 0; k < kVec; ++k) {
                qt[k] = w[k] * c.inv_s;
                alpha_loc += fminf(p[k], qt[k]);
                rsum += fmaxf(0.f, p[k] - qt[k]);
            }
            if (qrow) {
                if (qvec && base + kVec <= P.N) {
                    reinterpret_cast<float4*>(qrow + base)[0] = make_float4(qt[0], qt[1], qt[2], qt[3]);
                    reinterpret_cast<float4*>(qrow + base)[1] = make_float4(qt[4], qt[5], qt[6], qt[7]);
                } else {
#pragma unroll
                    for (int k = 0; k < kVec; ++k) if (base + k < P.N) qrow[base + k] = qt[k];
                }
            }
        }
        rsum = warp_sum(rsum);
        if (c.lane == 0) seg_r[tile * kRowWarps + c.warp] = rsum;
    }
    const double a_w = warp_sum_d((double)alpha_loc);
    if (c.lane == 0) red_a[c.warp] = a_w;
    __syncthreads();
    if (c.warp == 0) {
        const double tot = warp_scan_segments(seg_r, cdf_r, num_segs, c.lane);
        double a = (c.lane < kRowWarps) ? red_a[c.lane] : 0.0;
        a = warp_sum_d(a);
        if (c.lane == 0) { bc_d[1] = tot; bc[5] = (float)a; }
    }
    __syncthreads();
    const double R_d = bc_d[1];
    if (c.tid == 0) {
        if (P.alpha) P.alpha[row] = bc[5];
        if (P.theta) P.theta[row] = c.theta;
        if (P.S) P.S[row] = S;
        if (P.residual_mass) P.residual_mass[row] = (float)R_d;
    }

    // ---- draws: one warp per trial ---------------------------------------------------------------
    for (int t = c.warp; t < P.trials; t += kRowWarps) {
        const float* u = P.uniforms + ((long long)row * P.trials + t) * 4;
        const float u0 = __ldg(u), u1 = __ldg(u + 1), u2 = __ldg(u + 2);
        // draft token d ~ w / S
        const double thr = (double)u0 * S_d;
        int seg = first_above(cdf_w, num_segs, thr);
        if (seg >= num_segs) seg = num_segs - 1;
        float rem = (float)(thr - (seg ? cdf_w[seg - 1] : 0.0));
        int base = (seg / kRowWarps) * kTile + (seg % kRowWarps) * kSeg + c.lane * kVec;
        float p[kVec], w[kVec];
#pragma unroll
        for (int k = 0; k < kVec; ++k) { p[k] = 0.f; w[k] = 0.f; }
        if (base < P.N) load_pw<TZ, TY, MODE, KIND>(P, c, zrow, yrow, wrow, base, p, w);
        int sel = pick_in_segment(w, rem, c.lane);
        if (sel < 0) sel = 0;
        float pd = 0.f, wd = 0.f;
#pragma unroll
        for (int k = 0; k < kVec; ++k) if (k == (sel & (kVec - 1))) { pd = p[k]; wd = w[k]; }
        pd = __shfl_sync(0xffffffffu, pd, sel / kVec);
        wd = __shfl_sync(0xffffffffu, wd, sel / kVec);
        const int d = (seg / kRowWarps) * kTile + (seg % kRowWarps) * kSeg + sel;
        const float qd = wd * c.inv_s;
        const float a = (pd >= qd) ? 1.f : pd / qd;
        const bool acc = u1 * qd < pd;
        int out = d;
        if (!acc) {
            if (R_d > 0.0) {
                const double thr_r = (double)u2 * R_d;
                int sr = first_above(cdf_r, num_segs, thr_r);
                if (sr >= num_segs) sr = num_segs - 1;
                rem = (float)(thr_r - (sr ? cdf_r[sr - 1] : 0.0));
                base = (sr / kRowWarps) * kTile + (sr % kRowWarps) * kSeg + c.lane * kVec;
                float r[kVec];
#pragma unroll
                for (int k = 0; k < kVec; ++k) r[k] = 0.f;
                if (base < P.N) {
                    load_pw<TZ, TY, MODE, KIND>(P, c, zrow, yrow, wrow, base, p, w);
#pragma unroll
                    for (int k = 0; k < kVec; ++k) r[k] = fmaxf(0.f, p[k] - w[k] * c.inv_s);
                }
                int s2 = pick_in_segment(r, rem, c.lane);
                if (s2 < 0) s2 = 0;
                out = (sr / kRowWarps) * kTile + (sr % kRowWarps) * kSeg + s2;
            } else {
                // p and q~ coincide to rounding: the replacement is drawn from p itself
                const double thr_p = (double)u2;           // sum_j p_j = 1
                double run = 0.0;
                int last_seg = -1, last_sel = 0;
                out = -1;
                for (int s = 0; s < num_segs && out < 0; ++s) {
                    base = (s / kRowWarps) * kTile + (s % kRowWarps) * kSeg + c.lane * kVec;
#pragma unroll
                    for (int k = 0; k < kVec; ++k) p[k] = 0.f;
                    if (base < P.N) load_pw<TZ, TY, MODE, KIND>(P, c, zrow, yrow, wrow, base, p, w);
                    float ps = 0.f;
#pragma unroll
                    for (int k = 0; k < kVec; ++k) ps += p[k];
                    ps = warp_sum(ps);
                    if (ps > 0.f) {
                        last_seg = s;
                        if (run + (double)ps > thr_p) {
                            const int s3 = pick_in_segment(p, (float)(thr_p - run), c.lane);
                            out = (s / kRowWarps) * kTile + (s % kRowWarps) * kSeg + (s3 < 0 ? 0 : s3);
                        } else {
                            last_sel = pick_in_segment(p, INFINITY, c.lane);   // last positive token so far
                        }
                    }
                    run += (double)ps;
                }
                if (out < 0) out = last_seg < 0 ? 0 : (last_seg / kRowWarps) * kTile + (last_seg % kRowWarps) * kSeg + last_sel;
            }
        }
        if (c.lane == 0) {
            const long long o = (long long)row * P.trials + t;
            if (P.draft_token) P.draft_token[o] = d;
            if (P.out_token) P.out_token[o] = out;
            if (P.accepted) P.accepted[o] = acc ? 1 : 0;
            if (P.accept_prob) P.accept_prob[o] = a;
        }
    }
}

// accepted_len[b, t] = number of leading positions whose draft was accepted (Algorithm 4 step 7).
__global__ void accepted_len_kernel(const uint8_t* __restrict__ accepted, int32_t* __restrict__ out,
                                    int batch, int positions, int trials) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= batch * trials) return;
    const int b = g / trials, t = g % trials;
    int k = 0;
    while (k < positions && accepted[((long long)b * positions + k) * trials + t]) ++k;
    out[g] = k;
}

template <typename TZ, typename TY, int MODE>
static cudaError_t launch_kind(const RowParams& P, int kind, size_t smem, cudaStream_t s) {
    cudaError_t e;
    if (kind == RDK_LOGITS) {
        auto k = rdk_row_kernel<TZ, TY, MODE, RDK_LOGITS>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k<<<P.rows, kRowThreads, smem, s>>>(P);
    } else {
        auto k = rdk_row_kernel<TZ, TY, MODE, RDK_PROBS>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k<<<P.rows, kRowThreads, smem, s>>>(P);
    }
    return cudaGetLastError();
}

template <int MODE>
static cudaError_t launch_types(const RowParams& P, int tz, int ty, int kind, size_t smem, cudaStream_t s) {
    if (tz == RDK_F32) {
        if (ty == RDK_F32) return launch_kind<float, float, MODE>(P, kind, smem, s);
        return launch_kind<float, __nv_bfloat16, MODE>(P, kind, smem, s);
    }
    if (ty == RDK_F32) return launch_kind<__nv_bfloat16, float, MODE>(P, kind, smem, s);
    return launch_kind<__nv_bfloat16, __nv_bfloat16, MODE>(P, kind, smem, s);
}

constexpr int kMaxN = 1 << 21;   // the per-segment tables of one row must fit in shared memory

static int validate_problem(const rdk_problem* pb, const char* who, bool need_index) {
    if (!pb) { set_error("%s: problem is NULL", who); return RDK_ERR_INVALID_ARG; }
    if (pb->N < 1 || pb->n < 1 || pb->batch < 1 || pb->positions < 1) {
        set_error("%s: sizes must be positive (N=%d n=%d batch=%d positions=%d)", who, pb->N, pb->n, pb->batch, pb->positions);
        return RDK_ERR_INVALID_ARG;
    }
    if ((long long)pb->batch * pb->positions > 0x7fffffffLL) { set_error("%s: too many rows", who); return RDK_ERR_INVALID_ARG; }
    if ((pb->target_dtype != RDK_F32 && pb->target_dtype != RDK_BF16) ||
        (pb->drafter_dtype != RDK_F32 && pb->drafter_dtype != RDK_BF16) ||
        (pb->drafter_kind != RDK_LOGITS && pb->drafter_kind != RDK_PROBS) || (pb->flags & ~(RDK_FLAG_ROW_KERNEL | RDK_FLAG_W_AS_GIVEN)) != 0) {
        set_error("%s: bad dtype / kind / flags field", who);
        return RDK_ERR_INVALID_ARG;
    }
    if ((pb->target_row_stride != 0 && pb->target_row_stride < pb->N) ||
        (pb->drafter_row_stride != 0 && pb->drafter_row_stride < pb->n)) {
        set_error("%s: a row stride is smaller than the row", who);
        return RDK_ERR_INVALID_ARG;
    }
    if (need_index && !pb->kept_index) { set_error("%s: kept_index is NULL", who); return RDK_ERR_INVALID_ARG; }
    if (pb->N > kMaxN) { set_error("%s: N=%d exceeds the supported maximum %d", who, pb->N, kMaxN); return RDK_ERR_UNSUPPORTED; }
    return RDK_OK;
}

static int run_rows(const rdk_problem* pb, int mode, const void* target, const void* drafter,
                    const float* w, long long w_stride, const float* uniforms, int trials,
                    const rdk_outputs* out, float* qtilde, float* theta_out, float* S_out,
                    void* ws, size_t ws_bytes, cudaStream_t s, const void* prior = nullptr, long long prior_stride = 0) {
    RowParams P{};
    P.N = pb->N; P.n = pb->n; P.rows = pb->batch * pb->positions; P.trials = trials;
    P.target = target; P.target_stride = pb->target_row_stride ? pb->target_row_stride : pb->N;
    P.drafter = drafter; P.drafter_stride = pb->drafter_row_stride ? pb->drafter_row_stride : pb->n;
    P.w = w; P.w_stride = w_stride ? w_stride : pb->N;
    P.uniforms = uniforms;
    P.prior = prior; P.prior_stride = prior_stride;
    P.w_as_given = (pb->flags & RDK_FLAG_W_AS_GIVEN) ? 1 : 0;
    if (P.w_as_given && mode != RDK_MODE_PRECOMPUTED_W) {
        set_error("RDK_FLAG_W_AS_GIVEN applies to RDK_MODE_PRECOMPUTED_W only");
        return RDK_ERR_INVALID_ARG;
    }
    if (mode == RDK_MODE_LINEAR) {
        KeptIndexView v = make_view(pb->kept_index, pb->N, pb->n);
        P.header = v.header; P.mask = v.mask; P.rank = v.rank; P.slot = v.slot; P.ids = v.ids;
    }
    if (out) {
        P.draft_token = out->draft_token; P.out_token = out->out_token; P.accepted = out->accepted;
        P.accept_prob = out->accept_prob; P.alpha = out->alpha; P.theta = out->theta; P.S = out->S;
        P.residual_mass = out->residual_mass; P.status_word = out->status_word;
    }
    if (theta_out) P.theta = theta_out;
    if (S_out) P.S = S_out;
    P.qtilde = qtilde;
    P.num_tiles = (pb->N + kTile - 1) / kTile;
    const size_t smem = (size_t)P.num_tiles * kRowWarps * 24;
    cudaError_t e = cudaErrorNotSupported;
    P.positions = pb->positions;
    P.accepted_len = out ? out->accepted_len : nullptr;
    if (mode == RDK_MODE_LINEAR && trials > 0 && !prior && !(pb->flags & RDK_FLAG_ROW_KERNEL)) {
        e = launch_stream_linear(P, pb->target_dtype, pb->drafter_dtype, pb->drafter_kind, pb->batch, ws, ws_bytes, s);
        if (e == cudaSuccess) return RDK_OK;          // the streaming kernel also wrote accepted_len
    }
    if (e == cudaErrorNotSupported)
        e = (mode == RDK_MODE_LINEAR)
            ? launch_types<RDK_MODE_LINEAR>(P, pb->target_dtype, pb->drafter_dtype, pb->drafter_kind, smem, s)
            : launch_types<RDK_MODE_PRECOMPUTED_W>(P, pb->target_dtype, RDK_F32, RDK_LOGITS, smem, s);
    if (e != cudaSuccess) return cuda_fail(e, "row kernel launch");
    if (out && out->accepted_len && trials > 0) {
        if (!out->accepted) { set_error("accepted_len needs the accepted output"); return RDK_ERR_INVALID_ARG; }
        const int work = pb->batch * trials;
        accepted_len_kernel<<<(work + 127) / 128, 128, 0, s>>>(out->accepted, out->accepted_len, pb->batch, pb->positions, trials);
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "accepted_len kernel launch");
    }
    return RDK_OK;
}

}  // namespace rdk

using namespace rdk;

extern "C" int rdk_redistribute_linear(const rdk_problem* problem, const void* target, const void* drafter,
                                       float* qtilde_out, float* theta_out, float* S_out, void* stream) {
    int st = validate_problem(problem, "rdk_redistribute_linear", true);
    if (st != RDK_OK) return st;
    if (!target || !drafter || !qtilde_out) { set_error("rdk_redistribute_linear: null pointer"); return RDK_ERR_INVALID_ARG; }
    st = check_arch();
    if (st != RDK_OK) return st;
    return run_rows(problem, RDK_MODE_LINEAR, target, drafter, nullptr, 0, nullptr, 0, nullptr,
                    qtilde_out, theta_out, S_out, nullptr, 0, static_cast<cudaStream_t>(stream));
}

extern "C" int rdk_redistribute_linear_prior(const rdk_problem* problem, const void* target, const void* prior,
                                             int64_t prior_row_stride, const void* drafter, float* qtilde_out,
                                             float* theta_out, float* S_out, void* stream) {
    int st = validate_problem(problem, "rdk_redistribute_linear_prior", true);
    if (st != RDK_OK) return st;
    if (!target || !prior || !drafter || !qtilde_out || (prior_row_stride != 0 && prior_row_stride < problem->N)) {
        set_error("rdk_redistribute_linear_prior: null pointer or a prior row stride below N");
        return RDK_ERR_INVALID_ARG;
    }
    st = check_arch();
    if (st != RDK_OK) return st;
    return run_rows(problem, RDK_MODE_LINEAR, target, drafter, nullptr, 0, nullptr, 0, nullptr,
                    qtilde_out, theta_out, S_out, nullptr, 0, static_cast<cudaStream_t>(stream), prior, prior_row_stride);
}

extern "C" int rdk_sample_and_verify_prior(const rdk_problem* problem, const void* target, const void* prior,
                                           int64_t prior_row_stride, const void* drafter, const float* uniforms,
                                           int32_t trials, const rdk_outputs* out, void* stream) {
    int st = validate_problem(problem, "rdk_sample_and_verify_prior", true);
    if (st != RDK_OK) return st;
    if (!target || !prior || !drafter || !uniforms || !out || trials < 1 ||
        (prior_row_stride != 0 && prior_row_stride < problem->N)) {
        set_error("rdk_sample_and_verify_prior: null pointer, trials < 1 or a prior row stride below N");
        return RDK_ERR_INVALID_ARG;
    }
    if (out->accepted_len && !out->accepted) {
        set_error("rdk_sample_and_verify_prior: accepted_len needs the accepted output");
        return RDK_ERR_INVALID_ARG;
    }
    st = check_arch();
    if (st != RDK_OK) return st;
    return run_rows(problem, RDK_MODE_LINEAR, target, drafter, nullptr, 0, uniforms, trials, out, nullptr,
                    nullptr, nullptr, nullptr, 0, static_cast<cudaStream_t>(stream), prior, prior_row_stride);
}

extern "C" int rdk_sample_route(const rdk_problem* problem, int32_t mode, const void* target, const void* drafter,
                                int32_t trials, const void* ws, size_t ws_bytes, const char** why) {
    if (why) *why = "";
    int st = validate_problem(problem, "rdk_sample_route", mode == RDK_MODE_LINEAR);
    if (st != RDK_OK) return -st;
    if (mode != RDK_MODE_LINEAR) { if (why) *why = "precomputed w"; return RDK_ROUTE_ROW_KERNEL; }
    if (problem->flags & RDK_FLAG_W_AS_GIVEN) {
        set_error("RDK_FLAG_W_AS_GIVEN applies to RDK_MODE_PRECOMPUTED_W only");
        return -RDK_ERR_INVALID_ARG;
    }
    if (problem->flags & RDK_FLAG_ROW_KERNEL) { if (why) *why = "RDK_FLAG_ROW_KERNEL is set"; return RDK_ROUTE_ROW_KERNEL; }
    RowParams P{};
    P.N = problem->N; P.n = problem->n; P.rows = problem->batch * problem->positions; P.trials = trials;
    P.target = target; P.target_stride = problem->target_row_stride ? problem->target_row_stride : problem->N;
    P.drafter = drafter; P.drafter_stride = problem->drafter_row_stride ? problem->drafter_row_stride : problem->n;
    P.header = static_cast<const int32_t*>(problem->kept_index);
    const char* no = stream_ineligible(P, problem->target_dtype, problem->drafter_dtype, problem->drafter_kind,
                                       problem->batch, ws, ws_bytes);
    if (no) { if (why) *why = no; return RDK_ROUTE_ROW_KERNEL; }
    return RDK_ROUTE_STREAM_KERNEL;
}

extern "C" void rdk_test_set_spin_limit(uint32_t limit) { set_stream_spin_limit(limit); }

extern "C" size_t rdk_sample_workspace_bytes(const rdk_problem* problem, int32_t mode, int32_t trials) {
    if (!problem || mode != RDK_MODE_LINEAR || trials < 1 || problem->batch < 1 || problem->positions < 1) return 0;
    const long long rows = (long long)problem->batch * problem->positions;
    if (rows > 0x7fffffffLL) return 0;
    return stream_workspace_bytes((int)rows, problem->batch, trials);
}

extern "C" int rdk_sample_and_verify(const rdk_problem* problem, int32_t mode, const void* target,
                                     const void* drafter, const float* w, int64_t w_row_stride,
                                     const float* uniforms, int32_t trials, const rdk_outputs* out,
                                     void* ws, size_t ws_bytes, void* stream) {
    if (mode != RDK_MODE_LINEAR && mode != RDK_MODE_PRECOMPUTED_W) {
        set_error("rdk_sample_and_verify: unknown mode %d", mode);
        return RDK_ERR_INVALID_ARG;
    }
    int st = validate_problem(problem, "rdk_sample_and_verify", mode == RDK_MODE_LINEAR);
    if (st != RDK_OK) return st;
    if (!target || !uniforms || !out || trials < 1) {
        set_error("rdk_sample_and_verify: null pointer or trials < 1");
        return RDK_ERR_INVALID_ARG;
    }
    if (mode == RDK_MODE_LINEAR && (!drafter || w)) {
        set_error("rdk_sample_and_verify: linear mode needs drafter and w == NULL");
        return RDK_ERR_INVALID_ARG;
    }
    if (mode == RDK_MODE_PRECOMPUTED_W && (!w || (w_row_stride != 0 && w_row_stride < problem->N))) {
        set_error("rdk_sample_and_verify: precomputed mode needs w with a row stride >= N");
        return RDK_ERR_INVALID_ARG;
    }
    if (out->accepted_len && !out->accepted) {
        set_error("rdk_sample_and_verify: accepted_len needs the accepted output");
        return RDK_ERR_INVALID_ARG;
    }
    const size_t need = rdk_sample_workspace_bytes(problem, mode, trials);
    if (need > 0 && (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u))) {
        set_error("rdk_sample_and_verify: workspace of %zu bytes (256-byte aligned) needed, %zu given", need, ws ? ws_bytes : (size_t)0);
        return RDK_ERR_WORKSPACE_TOO_SMALL;
    }
    st = check_arch();
    if (st != RDK_OK) return st;
    return run_rows(problem, mode, target, drafter, w, w_row_stride, uniforms, trials, out, nullptr,
                    nullptr, nullptr, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

extern "C" int rdk_sample_and_verify_host(const rdk_problem* problem, const void* target_host,
                                          const void* drafter_host, const float* uniforms_host,
                                          int32_t trials, void* stage_target, void* stage_drafter,
                                          float* stage_uniforms, const rdk_outputs* dev_out,
                                          const rdk_outputs* host_out, void* ws, size_t ws_bytes, void* stream) {
    int st = validate_problem(problem, "rdk_sample_and_verify_host", true);
    if (st != RDK_OK) return st;
    if (!target_host || !drafter_host || !uniforms_host || !stage_target || !stage_drafter ||
        !stage_uniforms || !dev_out || !host_out || trials < 1) {
        set_error("rdk_sample_and_verify_host: null pointer or trials < 1");
        return RDK_ERR_INVALID_ARG;
    }
    if ((problem->target_row_stride != 0 && problem->target_row_stride != problem->N) ||
        (problem->drafter_row_stride != 0 && problem->drafter_row_stride != problem->n)) {
        set_error("rdk_sample_and_verify_host: host rows must be dense");
        return RDK_ERR_INVALID_ARG;
    }
    st = check_arch();
    if (st != RDK_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)problem->batch * problem->positions;
    const size_t zb = problem->target_dtype == RDK_F32 ? 4 : 2, yb = problem->drafter_dtype == RDK_F32 ? 4 : 2;
    RDK_CUDA(cudaMemcpyAsync(stage_target, target_host, rows * problem->N * zb, cudaMemcpyHostToDevice, s));
    RDK_CUDA(cudaMemcpyAsync(stage_drafter, drafter_host, rows * problem->n * yb, cudaMemcpyHostToDevice, s));
    RDK_CUDA(cudaMemcpyAsync(stage_uniforms, uniforms_host, rows * trials * 4 * sizeof(float), cudaMemcpyHostToDevice, s));
    st = rdk_sample_and_verify(problem, RDK_MODE_LINEAR, stage_target, stage_drafter, nullptr, 0,
                               stage_uniforms, trials, dev_out, ws, ws_bytes, stream);
    if (st != RDK_OK) return st;
    const size_t rt = rows * trials;
#define RDK_BACK(member, count, type)                                                             \
    if (dev_out->member && host_out->member)                                                      \
        RDK_CUDA(cudaMemcpyAsync(host_out->member, dev_out->member, (count) * sizeof(type), cudaMemcpyDeviceToHost, s));
    RDK_BACK(draft_token, rt, int32_t)
    RDK_BACK(out_token, rt, int32_t)
    RDK_BACK(accepted, rt, uint8_t)
    RDK_BACK(accept_prob, rt, float)
    RDK_BACK(alpha, rows, float)
    RDK_BACK(theta, rows, float)
    RDK_BACK(S, rows, float)
    RDK_BACK(residual_mass, rows, float)
    RDK_BACK(accepted_len, (size_t)problem->batch * trials, int32_t)
    RDK_BACK(status_word, 1, int32_t)
#undef RDK_BACK
    RDK_CUDA(cudaStreamSynchronize(s));
    return RDK_OK;
}
