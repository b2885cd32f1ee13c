// Token-affinity matrix (Eq. symbolic-m with Omega = cosine similarity) for bf16 embeddings and the bf16
// transposed layout, with the dot products on the tensor cores:
//   G[j, i] = <e_j, e_{kappa_i}>                       (bf16 x bf16 products are exact, fp32 accumulation;
//                                                       the tcgen05 kernel of the exact redistribution)
//   Mt[j, i] = exp((G[j, i] / (|e_j| |e_{kappa_i}|) - 1) / tau) / Z_i,
//   Z_i = sum_{j in T} exp((G[j, i] / (|e_j| |e_{kappa_i}|) - 1) / tau)
// (the shift by the largest possible cosine, 1, cancels in the quotient).  The kept rows are taken in chunks
// of at most kAffChunk; per chunk: gather the kept embeddings, one GEMM into an fp32 scratch [N, chunk],
// per-column sums in two deterministic steps, one pass that writes the bf16 result.
#include <math.h>

#include "rdk_common.cuh"

namespace rdk {

int launch_exact_tc(const __nv_bfloat16* A, long long lda, const __nv_bfloat16* Mt, long long ldm, float* w_out,
                    float* S_out, int rows, int n, int N, int32_t* status_word, cudaStream_t s);

constexpr int kAffChunk = 2048;          // kept rows per GEMM (columns of the fp32 scratch)
constexpr int kAffBlockRows = 64;        // token rows per CTA in the column-sum pass
constexpr int kAffColThreads = 256;

// inv[t] = 1 / max(|e_t|, 1e-12), one warp per token
__global__ void aff_inv_norm_kernel(const __nv_bfloat16* __restrict__ E, long long stride, float* __restrict__ inv, int N, int d) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N) return;
    const __nv_bfloat16* row = E + (long long)warp * stride;
    float ss = 0.f;
    for (int k = lane; k < d; k += 32) { const float v = __bfloat162float(row[k]); ss += v * v; }
    ss = warp_sum(ss);
    if (lane == 0) inv[warp] = 1.f / fmaxf(sqrtf(ss), 1e-12f);
}

// Ek[c, :] = e_{kappa_{i0 + c}} (zeros for an id outside [0, N)), invk[c] = its inverse norm (0 for such an id)
__global__ void aff_gather_kernel(const __nv_bfloat16* __restrict__ E, long long stride, const int32_t* __restrict__ ids,
                                  const float* __restrict__ inv, __nv_bfloat16* __restrict__ Ek, float* __restrict__ invk,
                                  int i0, int cols, int N, int d, int dpad) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= cols) return;
    const int id = ids[i0 + warp];
    const bool ok = id >= 0 && id < N;
    for (int k = lane; k < dpad; k += 32)
        Ek[(long long)warp * dpad + k] = (ok && k < d) ? E[(long long)id * stride + k] : __float2bfloat16_rn(0.f);
    if (lane == 0) invk[warp] = ok ? inv[id] : 0.f;
}

// part[b, c] = sum over the token rows j of block b of 2^((G[j, c] inv[j] invk[c] - 1) scale)
__global__ void __launch_bounds__(kAffColThreads)
aff_colsum_kernel(const float* __restrict__ G, const float* __restrict__ inv, const float* __restrict__ invk,
                  float* __restrict__ part, int N, int cols, float scale) {
    const int j0 = blockIdx.x * kAffBlockRows;
    const int j1 = min(N, j0 + kAffBlockRows);
    for (int c = threadIdx.x; c < cols; c += kAffColThreads) {
        const float ik = invk[c];
        float s = 0.f;
        for (int j = j0; j < j1; ++j)
            s += ex2((G[(long long)j * cols + c] * (__ldg(inv + j) * ik) - 1.f) * scale);
        part[(long long)blockIdx.x * cols + c] = s;
    }
}

// invZ[c] = 1 / sum_b part[b, c], blocks taken in order
__global__ void aff_colsum_reduce_kernel(const float* __restrict__ part, float* __restrict__ invZ, int blocks, int cols) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= cols) return;
    float s = 0.f;
    for (int b = 0; b < blocks; ++b) s += part[(long long)b * cols + c];
    invZ[c] = 1.f / s;
}

// Mt[j, i0 + c] = bf16(2^((G[j, c] inv[j] invk[c] - 1) scale) invZ[c]); kept ids outside the vocabulary give 0
__global__ void __launch_bounds__(kAffColThreads)
aff_write_kernel(const float* __restrict__ G, const float* __restrict__ inv, const float* __restrict__ invk,
                 const float* __restrict__ invZ, __nv_bfloat16* __restrict__ Mt, long long ld, int i0, int N, int cols, float scale) {
    const int j = blockIdx.x;
    const float ij = __ldg(inv + j);
    const float* g = G + (long long)j * cols;
    __nv_bfloat16* out = Mt + (long long)j * ld + i0;
    for (int c = threadIdx.x; c < cols; c += kAffColThreads) {
        const float ik = invk[c];
        const float v = ik > 0.f ? ex2((g[c] * (ij * ik) - 1.f) * scale) * invZ[c] : 0.f;
        out[c] = __float2bfloat16_rn(v);
    }
}

// a wait inside the tensor-core kernel ran out: the matrix is incomplete, make that impossible to miss
__global__ void aff_poison_kernel(const int32_t* status, __nv_bfloat16* Mt) {
    if (*status != 0) Mt[0] = __float2bfloat16_rn(NAN);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
static size_t aff_tc_dpad(int d) { return (size_t)((d + 7) & ~7); }
static int aff_tc_chunk(int n) { return n < kAffChunk ? n : kAffChunk; }

// workspace: inv[N] | invk[chunk] | invZ[chunk] | status | Ek[chunk, dpad] bf16 | part[blocks, chunk] | G[N, chunk]
struct AffTcLayout { size_t inv, invk, invZ, status, Ek, part, G, total; int chunk, blocks; };
static AffTcLayout aff_tc_layout(int N, int n, int d) {
    AffTcLayout L;
    L.chunk = aff_tc_chunk(n);
    L.blocks = (N + kAffBlockRows - 1) / kAffBlockRows;
    size_t o = 0;
    L.inv = o;    o += idx_align((size_t)N * sizeof(float));
    L.invk = o;   o += idx_align((size_t)L.chunk * sizeof(float));
    L.invZ = o;   o += idx_align((size_t)L.chunk * sizeof(float));
    L.status = o; o += idx_align(sizeof(int32_t));
    L.Ek = o;     o += idx_align((size_t)L.chunk * aff_tc_dpad(d) * sizeof(__nv_bfloat16));
    L.part = o;   o += idx_align((size_t)L.blocks * L.chunk * sizeof(float));
    L.G = o;      o += idx_align((size_t)N * L.chunk * sizeof(float));
    L.total = o;
    return L;
}

size_t affinity_tc_workspace_bytes(int N, int n, int d) { return aff_tc_layout(N, n, d).total; }

// whether the tensor-core route serves this call (the other route serves everything)
bool affinity_tc_eligible(const void* embeddings, int emb_dtype, int d, long long estride, int layout) {
    return emb_dtype == RDK_BF16 && layout == RDK_AFF_BF16_COLS && d >= 64 && (estride % 8) == 0 &&
           (reinterpret_cast<uintptr_t>(embeddings) & 15u) == 0;
}

int build_affinity_tc(const __nv_bfloat16* E, int d, long long estride, const int32_t* ids, int n, int N, float tau,
                      __nv_bfloat16* Mt, long long ld, void* ws, cudaStream_t s) {
    const AffTcLayout L = aff_tc_layout(N, n, d);
    unsigned char* base = static_cast<unsigned char*>(ws);
    float* inv = reinterpret_cast<float*>(base + L.inv);
    float* invk = reinterpret_cast<float*>(base + L.invk);
    float* invZ = reinterpret_cast<float*>(base + L.invZ);
    int32_t* status = reinterpret_cast<int32_t*>(base + L.status);
    __nv_bfloat16* Ek = reinterpret_cast<__nv_bfloat16*>(base + L.Ek);
    float* part = reinterpret_cast<float*>(base + L.part);
    float* G = reinterpret_cast<float*>(base + L.G);
    const int dpad = (int)aff_tc_dpad(d);
    const float scale = kLog2e / tau;
    const int wpb = 8;
    RDK_CUDA(cudaMemsetAsync(status, 0, sizeof(int32_t), s));
    aff_inv_norm_kernel<<<(N + wpb - 1) / wpb, wpb * 32, 0, s>>>(E, estride, inv, N, d);
    RDK_CUDA(cudaGetLastError());
    for (int i0 = 0; i0 < n; i0 += L.chunk) {
        const int cols = n - i0 < L.chunk ? n - i0 : L.chunk;
        aff_gather_kernel<<<(cols + wpb - 1) / wpb, wpb * 32, 0, s>>>(E, estride, ids, inv, Ek, invk, i0, cols, N, d, dpad);
        RDK_CUDA(cudaGetLastError());
        // G[j, c] = sum_k E[j, k] Ek[c, k]: the GEMM of the exact redistribution with the roles
        // (rows, contraction, columns) = (tokens, embedding dimension, kept rows of the chunk)
        const int st = launch_exact_tc(E, estride, Ek, dpad, G, nullptr, N, d, cols, status, s);
        if (st != RDK_OK) return st;
        aff_colsum_kernel<<<L.blocks, kAffColThreads, 0, s>>>(G, inv, invk, part, N, cols, scale);
        RDK_CUDA(cudaGetLastError());
        aff_colsum_reduce_kernel<<<(cols + 127) / 128, 128, 0, s>>>(part, invZ, L.blocks, cols);
        RDK_CUDA(cudaGetLastError());
        aff_write_kernel<<<N, kAffColThreads, 0, s>>>(G, inv, invk, invZ, Mt, ld, i0, N, cols, scale);
        RDK_CUDA(cudaGetLastError());
    }
    aff_poison_kernel<<<1, 1, 0, s>>>(status, Mt);
    RDK_CUDA(cudaGetLastError());
    return RDK_OK;
}

}  // namespace rdk
