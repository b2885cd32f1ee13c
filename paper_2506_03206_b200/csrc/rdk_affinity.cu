// Token-affinity matrix, Eq. symbolic-m with Omega = cosine similarity of token embeddings:
//   M_ij = exp(Omega_ij / tau) / sum_{k in T} exp(Omega_ik / tau),  i in I (kept ids), j in T.
// One-time preprocessing: fp32 FMAs, two sweeps over the columns per block of kept rows
// (running max / sum first, normalised values second).
#include <math.h>

#include "rdk_common.cuh"

namespace rdk {

constexpr int kAffRows = 16;      // kept rows per CTA
constexpr int kAffThreads = 256;

// Et[k * N + t] = e_t[k] / max(|e_t|, 1e-12): unit-length embeddings, stored dimension-major so
// that consecutive threads (tokens) read consecutive addresses.
template <typename TE>
__global__ void aff_normalise_kernel(const TE* __restrict__ E, long long stride, float* __restrict__ Et, int N, int d) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N) return;
    const TE* row = E + (long long)warp * stride;
    float ss = 0.f;
    for (int k = lane; k < d; k += 32) { const float v = to_float<TE>(row[k]); ss += v * v; }
    ss = warp_sum(ss);
    const float inv = 1.f / fmaxf(sqrtf(ss), 1e-12f);
    for (int k = lane; k < d; k += 32) Et[(long long)k * N + warp] = to_float<TE>(row[k]) * inv;
}

template <int LAYOUT>
__global__ void __launch_bounds__(kAffThreads)
aff_rows_kernel(const float* __restrict__ Et, const int32_t* __restrict__ ids, int N, int n, int d,
                float scale /* log2(e) / tau */, void* __restrict__ Mout, long long ld) {
    extern __shared__ __align__(16) float rows_s[];          // [d][kAffRows]
    __shared__ float red_m[kAffThreads / 32][kAffRows], red_s[kAffThreads / 32][kAffRows];
    __shared__ float fin_m[kAffRows], fin_inv[kAffRows];
    __shared__ int id_s[kAffRows];
    const int i0 = blockIdx.x * kAffRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < kAffRows) {
        const int i = i0 + tid;
        const int id = (i < n) ? ids[i] : -1;
        id_s[tid] = (id >= 0 && id < N) ? id : -1;
    }
    __syncthreads();
    for (int x = tid; x < d * kAffRows; x += kAffThreads) {
        const int k = x / kAffRows, r = x % kAffRows;
        rows_s[x] = id_s[r] >= 0 ? Et[(long long)k * N + id_s[r]] : 0.f;
    }
    __syncthreads();

    float m[kAffRows], s[kAffRows];
#pragma unroll
    for (int r = 0; r < kAffRows; ++r) { m[r] = -INFINITY; s[r] = 0.f; }

    for (int pass = 0; pass < 2; ++pass) {
        for (int j = tid; j < N; j += kAffThreads) {
            float acc[kAffRows];
#pragma unroll
            for (int r = 0; r < kAffRows; ++r) acc[r] = 0.f;
            for (int k = 0; k < d; ++k) {
                const float a = __ldg(Et + (long long)k * N + j);
                const float4* rv = reinterpret_cast<const float4*>(rows_s + k * kAffRows);
#pragma unroll
                for (int q = 0; q < kAffRows / 4; ++q) {
                    const float4 b = rv[q];
                    acc[4 * q + 0] = fmaf(a, b.x, acc[4 * q + 0]);
                    acc[4 * q + 1] = fmaf(a, b.y, acc[4 * q + 1]);
                    acc[4 * q + 2] = fmaf(a, b.z, acc[4 * q + 2]);
                    acc[4 * q + 3] = fmaf(a, b.w, acc[4 * q + 3]);
                }
            }
            if (pass == 0) {
#pragma unroll
                for (int r = 0; r < kAffRows; ++r) {
                    const float x = acc[r] * scale;                    // Omega_ij / tau in base-2 units
                    if (x > m[r]) { s[r] = s[r] * ex2(m[r] - x) + 1.f; m[r] = x; }
                    else s[r] += ex2(x - m[r]);
                }
            } else {
                if (LAYOUT == RDK_AFF_F32_ROWS) {
                    float* M = static_cast<float*>(Mout);
#pragma unroll
                    for (int r = 0; r < kAffRows; ++r)
                        if (i0 + r < n) M[(long long)(i0 + r) * ld + j] = id_s[r] >= 0 ? ex2(fmaf(acc[r], scale, -fin_m[r])) * fin_inv[r] : 0.f;
                } else {
                    __nv_bfloat16* Mt = static_cast<__nv_bfloat16*>(Mout) + (long long)j * ld + i0;
#pragma unroll
                    for (int r = 0; r < kAffRows; ++r)
                        if (i0 + r < n) Mt[r] = __float2bfloat16_rn(id_s[r] >= 0 ? ex2(fmaf(acc[r], scale, -fin_m[r])) * fin_inv[r] : 0.f);
                }
            }
        }
        if (pass == 0) {
#pragma unroll
            for (int r = 0; r < kAffRows; ++r) {
                float mm = warp_max(m[r]);
                float ssum = (m[r] == -INFINITY) ? 0.f : s[r] * ex2(m[r] - mm);
                ssum = warp_sum(ssum);
                if (lane == 0) { red_m[warp][r] = mm; red_s[warp][r] = ssum; }
            }
            __syncthreads();
            if (tid < kAffRows) {
                float mm = -INFINITY;
                for (int w = 0; w < kAffThreads / 32; ++w) mm = fmaxf(mm, red_m[w][tid]);
                float ssum = 0.f;
                for (int w = 0; w < kAffThreads / 32; ++w)
                    if (red_m[w][tid] > -INFINITY) ssum += red_s[w][tid] * ex2(red_m[w][tid] - mm);
                fin_m[tid] = mm;
                fin_inv[tid] = 1.f / ssum;
            }
            __syncthreads();
        }
    }
}

// the tensor-core route (bf16 embeddings into the bf16 layout)
size_t affinity_tc_workspace_bytes(int N, int n, int d);
bool affinity_tc_eligible(const void* embeddings, int emb_dtype, int d, long long estride, int layout);
int build_affinity_tc(const __nv_bfloat16* E, int d, long long estride, const int32_t* ids, int n, int N, float tau,
                      __nv_bfloat16* Mt, long long ld, void* ws, cudaStream_t s);

}  // namespace rdk

using namespace rdk;

extern "C" size_t rdk_build_affinity_workspace_bytes(int32_t N, int32_t n, int32_t d) {
    if (N < 1 || n < 1 || d < 1) return 0;
    const size_t fma = idx_align((size_t)N * d * sizeof(float)), tc = affinity_tc_workspace_bytes(N, n, d);
    return fma > tc ? fma : tc;          // either route may serve the call
}

extern "C" int rdk_build_affinity(const void* embeddings, int32_t emb_dtype, int32_t d, int64_t emb_row_stride,
                                  const int32_t* kept_ids, int32_t n, int32_t N, float tau,
                                  const rdk_affinity* M_desc, void* M_out, void* ws, size_t ws_bytes,
                                  void* stream) {
    if (!embeddings || !kept_ids || !M_desc || !M_out || !ws || N < 1 || n < 1 || d < 1 || !(tau > 0.f)) {
        set_error("rdk_build_affinity: null pointer, non-positive size or tau <= 0");
        return RDK_ERR_INVALID_ARG;
    }
    if (emb_dtype != RDK_F32 && emb_dtype != RDK_BF16) { set_error("rdk_build_affinity: bad embedding dtype"); return RDK_ERR_INVALID_ARG; }
    const long long estride = emb_row_stride ? emb_row_stride : d;
    if (estride < d) { set_error("rdk_build_affinity: embedding row stride smaller than d"); return RDK_ERR_INVALID_ARG; }
    if (M_desc->reserved != 0) { set_error("rdk_build_affinity: reserved field must be 0"); return RDK_ERR_INVALID_ARG; }
    if (M_desc->layout == RDK_AFF_F32_ROWS) {
        if (M_desc->ld < N) { set_error("rdk_build_affinity: ld < N"); return RDK_ERR_INVALID_ARG; }
    } else if (M_desc->layout == RDK_AFF_BF16_COLS) {
        if (M_desc->ld < n || (M_desc->ld % 8) != 0 || (reinterpret_cast<uintptr_t>(M_out) & 15u)) {
            set_error("rdk_build_affinity: bf16 layout needs ld >= n, ld %% 8 == 0 and a 16-byte aligned base");
            return RDK_ERR_INVALID_ARG;
        }
    } else {
        set_error("rdk_build_affinity: unknown layout %d", M_desc->layout);
        return RDK_ERR_INVALID_ARG;
    }
    if (ws_bytes < rdk_build_affinity_workspace_bytes(N, n, d)) {
        set_error("rdk_build_affinity: workspace has %zu bytes, %zu needed", ws_bytes, rdk_build_affinity_workspace_bytes(N, n, d));
        return RDK_ERR_WORKSPACE_TOO_SMALL;
    }
    const size_t smem = (size_t)d * kAffRows * sizeof(float);
    if (smem > 200 * 1024) { set_error("rdk_build_affinity: embedding dimension %d too large", d); return RDK_ERR_UNSUPPORTED; }
    const int st = check_arch();
    if (st != RDK_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (affinity_tc_eligible(embeddings, emb_dtype, d, estride, M_desc->layout))
        return build_affinity_tc(static_cast<const __nv_bfloat16*>(embeddings), d, estride, kept_ids, n, N, tau,
                                 static_cast<__nv_bfloat16*>(M_out), M_desc->ld, ws, s);
    float* Et = static_cast<float*>(ws);
    const int wpb = 8;
    if (emb_dtype == RDK_F32)
        aff_normalise_kernel<float><<<(N + wpb - 1) / wpb, wpb * 32, 0, s>>>(static_cast<const float*>(embeddings), estride, Et, N, d);
    else
        aff_normalise_kernel<__nv_bfloat16><<<(N + wpb - 1) / wpb, wpb * 32, 0, s>>>(static_cast<const __nv_bfloat16*>(embeddings), estride, Et, N, d);
    RDK_CUDA(cudaGetLastError());
    const float scale = kLog2e / tau;
    const int blocks = (n + kAffRows - 1) / kAffRows;
    if (M_desc->layout == RDK_AFF_F32_ROWS) {
        RDK_CUDA(cudaFuncSetAttribute(aff_rows_kernel<RDK_AFF_F32_ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        aff_rows_kernel<RDK_AFF_F32_ROWS><<<blocks, kAffThreads, smem, s>>>(Et, kept_ids, N, n, d, scale, M_out, M_desc->ld);
    } else {
        RDK_CUDA(cudaFuncSetAttribute(aff_rows_kernel<RDK_AFF_BF16_COLS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        aff_rows_kernel<RDK_AFF_BF16_COLS><<<blocks, kAffThreads, smem, s>>>(Et, kept_ids, N, n, d, scale, M_out, M_desc->ld);
    }
    RDK_CUDA(cudaGetLastError());
    return RDK_OK;
}
