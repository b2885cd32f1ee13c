// Exact redistribution, Algorithm 1 steps 1-2:  q' = TLI(softmax(y)),  w = M^T q'.
// This file holds the operand preparation (q' at the kept slots), the fp32 FMA contraction for
// the fp32 row layout of M, the row sums S, and the entry point; the tensor-core contraction for
// the bf16 layout lives in rdk_exact_tc.cu.
#include <math.h>

#include "rdk_common.cuh"

namespace rdk {

int launch_exact_tc(const __nv_bfloat16* A, long long lda, const __nv_bfloat16* Mt, long long ldm,
                    float* w_out, float* S_out, int rows, int n, int N, int32_t* status_word, cudaStream_t s);

// A[r, i] = q'_{kappa_i}: soft-max over the drafter entries whose id lies in the target vocabulary
// (Eq. tli-drafter: drop the rest, renormalise), zero for dropped entries and for the padding
// columns i in [n, lda).
template <typename TY, typename TA, int KIND>
__global__ void __launch_bounds__(256)
exact_operand_kernel(const TY* __restrict__ drafter, long long dstride, const int32_t* __restrict__ ids,
                     int N, int n, TA* __restrict__ A, long long lda) {
    __shared__ float red[8];
    __shared__ float bc[2];
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TY* y = drafter + (long long)row * dstride;
    float m = -INFINITY;
    if (KIND == RDK_LOGITS) {
        for (int i = tid; i < n; i += 256) {
            const int id = ids[i];
            if (id >= 0 && id < N) m = fmaxf(m, to_float<TY>(y[i]));
        }
        m = warp_max(m);
        if (lane == 0) red[warp] = m;
        __syncthreads();
        if (tid == 0) { float mm = red[0]; for (int k = 1; k < 8; ++k) mm = fmaxf(mm, red[k]); bc[0] = mm; }
        __syncthreads();
        m = bc[0];
    }
    float s = 0.f;
    for (int i = tid; i < n; i += 256) {
        const int id = ids[i];
        if (id >= 0 && id < N) {
            const float v = to_float<TY>(y[i]);
            s += (KIND == RDK_LOGITS) ? ex2((v - m) * kLog2e) : v;
        }
    }
    s = warp_sum(s);
    __syncthreads();
    if (lane == 0) red[warp] = s;
    __syncthreads();
    if (tid == 0) { float t = 0.f; for (int k = 0; k < 8; ++k) t += red[k]; bc[1] = 1.f / t; }
    __syncthreads();
    const float inv = bc[1];
    TA* a = A + (long long)row * lda;
    for (int i = tid; i < lda; i += 256) {
        float q = 0.f;
        if (i < n) {
            const int id = ids[i];
            if (id >= 0 && id < N) {
                const float v = to_float<TY>(y[i]);
                q = ((KIND == RDK_LOGITS) ? ex2((v - m) * kLog2e) : v) * inv;
            }
        }
        if (sizeof(TA) == 4) reinterpret_cast<float*>(a)[i] = q;
        else reinterpret_cast<__nv_bfloat16*>(a)[i] = __float2bfloat16_rn(q);
    }
}

constexpr int kSimtRows = 8;

// w[r, j] = sum_i A[r, i] M[i, j]  with fp32 FMAs (fp32 row layout of M; small problems).
__global__ void __launch_bounds__(256)
exact_simt_kernel(const float* __restrict__ A, long long lda, const float* __restrict__ M, long long ldm,
                  float* __restrict__ w, int rows, int n, int N) {
    __shared__ float a_s[kSimtRows][256];
    const int j = blockIdx.x * 256 + threadIdx.x;
    const int r0 = blockIdx.y * kSimtRows;
    float acc[kSimtRows];
#pragma unroll
    for (int r = 0; r < kSimtRows; ++r) acc[r] = 0.f;
    for (int i0 = 0; i0 < n; i0 += 256) {
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSimtRows; ++r) {
            const int i = i0 + threadIdx.x;
            a_s[r][threadIdx.x] = (r0 + r < rows && i < n) ? A[(long long)(r0 + r) * lda + i] : 0.f;
        }
        __syncthreads();
        if (j < N) {
            const int lim = min(256, n - i0);
            for (int ii = 0; ii < lim; ++ii) {
                const float mv = __ldg(M + (long long)(i0 + ii) * ldm + j);
#pragma unroll
                for (int r = 0; r < kSimtRows; ++r) acc[r] = fmaf(a_s[r][ii], mv, acc[r]);
            }
        }
    }
    if (j < N) {
#pragma unroll
        for (int r = 0; r < kSimtRows; ++r)
            if (r0 + r < rows) w[(long long)(r0 + r) * N + j] = acc[r];
    }
}

// S[r] = sum_j w[r, j]
__global__ void __launch_bounds__(256)
row_sum_kernel(const float* __restrict__ w, int N, float* __restrict__ S) {
    __shared__ double red[8];
    const float* row = w + (long long)blockIdx.x * N;
    float s = 0.f;
    double acc = 0.0;
    int cnt = 0;
    for (int j = threadIdx.x; j < N; j += 256) {
        s += row[j];
        if (++cnt == 64) { acc += (double)s; s = 0.f; cnt = 0; }
    }
    acc += (double)s;
    acc = warp_sum_d(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) { double t = 0.0; for (int k = 0; k < 8; ++k) t += red[k]; S[blockIdx.x] = (float)t; }
}

template <typename TY, typename TA>
static void launch_operand(const void* drafter, long long dstride, const int32_t* ids, int N, int n, int kind,
                           void* A, long long lda, int rows, cudaStream_t s) {
    if (kind == RDK_LOGITS)
        exact_operand_kernel<TY, TA, RDK_LOGITS><<<rows, 256, 0, s>>>(static_cast<const TY*>(drafter), dstride, ids, N, n, static_cast<TA*>(A), lda);
    else
        exact_operand_kernel<TY, TA, RDK_PROBS><<<rows, 256, 0, s>>>(static_cast<const TY*>(drafter), dstride, ids, N, n, static_cast<TA*>(A), lda);
}

static long long operand_ld(int n, int layout) {
    return layout == RDK_AFF_BF16_COLS ? ((n + 63) / 64) * 64LL : n;
}

}  // namespace rdk

using namespace rdk;

extern "C" size_t rdk_exact_workspace_bytes(const rdk_problem* problem, int32_t affinity_layout) {
    if (!problem || problem->n < 1 || problem->batch < 1 || problem->positions < 1) return 0;
    if (affinity_layout != RDK_AFF_F32_ROWS && affinity_layout != RDK_AFF_BF16_COLS) return 0;
    const size_t rows = (size_t)problem->batch * problem->positions;
    const size_t el = affinity_layout == RDK_AFF_BF16_COLS ? 2 : 4;
    return idx_align(rows * (size_t)operand_ld(problem->n, affinity_layout) * el);
}

extern "C" int rdk_redistribute_exact(const rdk_problem* problem, const void* drafter, const rdk_affinity* M,
                                      float* w_out, float* S_out, void* ws, size_t ws_bytes,
                                      int32_t* status_word, void* stream) {
    if (!problem || !drafter || !M || !M->data || !w_out || !ws) {
        set_error("rdk_redistribute_exact: null pointer");
        return RDK_ERR_INVALID_ARG;
    }
    if (problem->N < 1 || problem->n < 1 || problem->batch < 1 || problem->positions < 1 || !problem->kept_index ||
        (problem->drafter_dtype != RDK_F32 && problem->drafter_dtype != RDK_BF16) ||
        (problem->drafter_kind != RDK_LOGITS && problem->drafter_kind != RDK_PROBS) || (problem->flags & ~(RDK_FLAG_ROW_KERNEL | RDK_FLAG_W_AS_GIVEN)) != 0 ||
        (problem->drafter_row_stride != 0 && problem->drafter_row_stride < problem->n) || M->reserved != 0) {
        set_error("rdk_redistribute_exact: bad problem description");
        return RDK_ERR_INVALID_ARG;
    }
    const int N = problem->N, n = problem->n;
    const long long rows_ll = (long long)problem->batch * problem->positions;
    if (rows_ll > 0x7fffffffLL) { set_error("rdk_redistribute_exact: too many rows"); return RDK_ERR_INVALID_ARG; }
    const int rows = (int)rows_ll;
    if (M->layout == RDK_AFF_F32_ROWS) {
        if (M->ld < N) { set_error("rdk_redistribute_exact: ld < N"); return RDK_ERR_INVALID_ARG; }
    } else if (M->layout == RDK_AFF_BF16_COLS) {
        if (M->ld < n || (M->ld % 8) != 0 || (reinterpret_cast<uintptr_t>(M->data) & 15u)) {
            set_error("rdk_redistribute_exact: bf16 layout needs ld >= n, ld %% 8 == 0 and a 16-byte aligned base");
            return RDK_ERR_INVALID_ARG;
        }
    } else {
        set_error("rdk_redistribute_exact: unknown affinity layout %d", M->layout);
        return RDK_ERR_INVALID_ARG;
    }
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) { set_error("rdk_redistribute_exact: workspace must be 256-byte aligned"); return RDK_ERR_INVALID_ARG; }
    if (ws_bytes < rdk_exact_workspace_bytes(problem, M->layout)) {
        set_error("rdk_redistribute_exact: workspace has %zu bytes, %zu needed", ws_bytes, rdk_exact_workspace_bytes(problem, M->layout));
        return RDK_ERR_WORKSPACE_TOO_SMALL;
    }
    int st = check_arch();
    if (st != RDK_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    KeptIndexView v = make_view(problem->kept_index, N, n);
    const long long dstride = problem->drafter_row_stride ? problem->drafter_row_stride : n;
    const long long lda = operand_ld(n, M->layout);
    const bool bf = M->layout == RDK_AFF_BF16_COLS;
    if (problem->drafter_dtype == RDK_F32) {
        if (bf) launch_operand<float, __nv_bfloat16>(drafter, dstride, v.ids, N, n, problem->drafter_kind, ws, lda, rows, s);
        else launch_operand<float, float>(drafter, dstride, v.ids, N, n, problem->drafter_kind, ws, lda, rows, s);
    } else {
        if (bf) launch_operand<__nv_bfloat16, __nv_bfloat16>(drafter, dstride, v.ids, N, n, problem->drafter_kind, ws, lda, rows, s);
        else launch_operand<__nv_bfloat16, float>(drafter, dstride, v.ids, N, n, problem->drafter_kind, ws, lda, rows, s);
    }
    RDK_CUDA(cudaGetLastError());
    if (bf) {
        // the tensor-core epilogue also accumulates S (one atomic partial sum per row and tile)
        return launch_exact_tc(static_cast<const __nv_bfloat16*>(ws), lda, static_cast<const __nv_bfloat16*>(M->data), M->ld,
                               w_out, S_out, rows, n, N, status_word, s);
    } else {
        dim3 grid((N + 255) / 256, (rows + kSimtRows - 1) / kSimtRows);
        exact_simt_kernel<<<grid, 256, 0, s>>>(static_cast<const float*>(ws), lda, static_cast<const float*>(M->data), M->ld, w_out, rows, n, N);
        RDK_CUDA(cudaGetLastError());
    }
    if (S_out) {
        row_sum_kernel<<<rows, 256, 0, s>>>(w_out, N, S_out);
        RDK_CUDA(cudaGetLastError());
    }
    return RDK_OK;
}

// ------------------------------------------------------------------------------------------------
// Variant of rdk_redistribute_exact whose q' operand lives in a fixed device array instead of a
// caller-supplied workspace, for callers that are not able to allocate device memory.
// ------------------------------------------------------------------------------------------------
#include <mutex>

static __device__ __align__(256) unsigned char g_exact_static_scratch[RDK_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {nullptr};
}  // namespace

extern "C" int rdk_redistribute_exact_static(const rdk_problem* problem, const void* drafter,
                                             const rdk_affinity* M, float* w_out, float* S_out,
                                             int32_t* status_word, void* stream) {
    if (!problem || !M) {
        set_error("rdk_redistribute_exact_static: null pointer");
        return RDK_ERR_INVALID_ARG;
    }
    const size_t need = rdk_exact_workspace_bytes(problem, M->layout);
    if (need == 0) {
        set_error("rdk_redistribute_exact_static: bad sizes or affinity layout");
        return RDK_ERR_INVALID_ARG;
    }
    if (need > (size_t)RDK_STATIC_SCRATCH_BYTES) {
        set_error("rdk_redistribute_exact_static: the q' operand needs %zu bytes but the built-in scratch array holds "
                  "%zu; use rdk_redistribute_exact with your own workspace", need, (size_t)RDK_STATIC_SCRATCH_BYTES);
        return RDK_ERR_WORKSPACE_TOO_SMALL;
    }
    int dev = 0;
    RDK_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error("rdk_redistribute_exact_static: device ordinal %d not supported", dev);
        return RDK_ERR_UNSUPPORTED;
    }
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_ptr[dev]) {
            // The array's name is only a host-side handle; the kernels need its device address.
            void* p = nullptr;
            RDK_CUDA(cudaGetSymbolAddress(&p, g_exact_static_scratch));
            g_scratch_ptr[dev] = p;
        }
        scratch = g_scratch_ptr[dev];
    }
    // Every element of the operand that the contraction reads is written first by the operand
    // kernel (padding columns included), so nothing left over from an earlier call is ever used.
    return rdk_redistribute_exact(problem, drafter, M, w_out, S_out, scratch, (size_t)RDK_STATIC_SCRATCH_BYTES,
                                  status_word, stream);
}
