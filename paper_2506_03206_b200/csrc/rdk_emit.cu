// Emitted sequences, Algorithm 4 steps 7-9: for every sequence (and trial) the accepted drafts
// d_1..d_j followed by one more token t -- the residual draw of the first rejected position, or,
// when all drafts were accepted, a fresh draw t ~ p from the target row that follows the last draft
// (inverse CDF in ascending token id with uniform lane 3 of the sequence's last position).
#include "rdk_row.cuh"

namespace rdk {

constexpr int kEmitThreads = 256;
constexpr int kEmitWarps = kEmitThreads / 32;
constexpr int kEmitTile = kEmitThreads * kVec;

struct EmitParams {
    int N, batch, positions, trials, num_tiles;
    const void* bonus; long long bonus_stride;
    const float* uniforms;
    const int32_t* draft_token; const uint8_t* accepted; const int32_t* out_token;
    int32_t* seq_tokens; int32_t* seq_len;
};

template <typename TZ>
__global__ void __launch_bounds__(kEmitThreads)
emit_kernel(const EmitParams P) {
    extern __shared__ __align__(16) unsigned char emit_smem[];
    const int num_segs = P.num_tiles * kEmitWarps;
    double* cdf = reinterpret_cast<double*>(emit_smem);
    float* seg = reinterpret_cast<float*>(cdf + num_segs);
    __shared__ MS red[kEmitWarps];
    __shared__ float bc[2];
    __shared__ double tot_s;
    __shared__ int j_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / P.trials, t = blockIdx.x % P.trials;
    if (tid == 0) {
        int j = 0;
        while (j < P.positions && P.accepted[((long long)b * P.positions + j) * P.trials + t]) ++j;
        j_s = j;
    }
    __syncthreads();
    const int j = j_s;
    int32_t* seq = P.seq_tokens + ((long long)b * P.trials + t) * (P.positions + 1);
    for (int k = tid; k < j; k += kEmitThreads) seq[k] = P.draft_token[((long long)b * P.positions + k) * P.trials + t];
    if (tid == 0) P.seq_len[(long long)b * P.trials + t] = j + 1;
    if (j < P.positions) {       // the residual draw made at the first rejected position
        if (tid == 0) seq[j] = P.out_token[((long long)b * P.positions + j) * P.trials + t];
        return;
    }

    // every draft accepted: t ~ softmax(bonus row)
    const TZ* zrow = static_cast<const TZ*>(P.bonus) + (long long)b * P.bonus_stride;
    const bool zvec = (reinterpret_cast<uintptr_t>(zrow) & 15u) == 0;
    MS zs{-INFINITY, 0.f, 0.f};
    for (int tile = 0; tile < P.num_tiles; ++tile) {
        const int base = tile * kEmitTile + tid * kVec;
        if (base >= P.N) break;
        float z[kVec];
        load8<TZ>(zrow, base, P.N, zvec, -INFINITY, z);
        float vmax = z[0];
#pragma unroll
        for (int k = 1; k < kVec; ++k) vmax = fmaxf(vmax, z[k]);
        if (vmax == -INFINITY) continue;
        if (vmax > zs.m) { zs.s *= ex2((zs.m - vmax) * kLog2e); zs.m = vmax; }
        const float off = -zs.m * kLog2e;
#pragma unroll
        for (int k = 0; k < kVec; ++k) zs.s += ex2(fmaf(z[k], kLog2e, off));
    }
    zs = ms_warp(zs);
    if (lane == 0) red[warp] = zs;
    __syncthreads();
    if (warp == 0) {
        MS a = lane < kEmitWarps ? red[lane] : MS{-INFINITY, 0.f, 0.f};
        a = ms_warp(a);
        if (lane == 0) { bc[0] = -a.m * kLog2e; bc[1] = 1.f / a.s; }
    }
    __syncthreads();
    const float off = bc[0], inv_z = bc[1];
    for (int tile = 0; tile < P.num_tiles; ++tile) {
        const int base = tile * kEmitTile + tid * kVec;
        float sum = 0.f;
        if (base < P.N) {
            float z[kVec];
            load8<TZ>(zrow, base, P.N, zvec, -INFINITY, z);
#pragma unroll
            for (int k = 0; k < kVec; ++k) sum += ex2(fmaf(z[k], kLog2e, off)) * inv_z;
        }
        sum = warp_sum(sum);
        if (lane == 0) seg[tile * kEmitWarps + warp] = sum;
    }
    __syncthreads();
    if (warp == 0) {
        const double tot = warp_scan_segments(seg, cdf, num_segs, lane);
        if (lane == 0) tot_s = tot;
    }
    __syncthreads();
    if (warp == 0) {
        const float u = __ldg(P.uniforms + (((long long)b * P.positions + P.positions - 1) * P.trials + t) * 4 + 3);
        const double thr = (double)u * tot_s;
        int s = first_above(cdf, num_segs, thr);
        if (s >= num_segs) s = num_segs - 1;
        const float rem = (float)(thr - (s ? cdf[s - 1] : 0.0));
        const int base = (s / kEmitWarps) * kEmitTile + (s % kEmitWarps) * kSeg + lane * kVec;
        float p[kVec];
#pragma unroll
        for (int k = 0; k < kVec; ++k) p[k] = 0.f;
        if (base < P.N) {
            float z[kVec];
            load8<TZ>(zrow, base, P.N, zvec, -INFINITY, z);
#pragma unroll
            for (int k = 0; k < kVec; ++k) p[k] = ex2(fmaf(z[k], kLog2e, off)) * inv_z;
        }
        int sel = pick_in_segment(p, rem, lane);
        if (sel < 0) sel = 0;
        if (lane == 0) seq[j] = (s / kEmitWarps) * kEmitTile + (s % kEmitWarps) * kSeg + sel;
    }
}

}  // namespace rdk

using namespace rdk;

extern "C" int rdk_emit_sequences(const rdk_problem* problem, const void* bonus_target, int64_t bonus_row_stride,
                                  const float* uniforms, int32_t trials, const int32_t* draft_token,
                                  const uint8_t* accepted, const int32_t* out_token, int32_t* seq_tokens,
                                  int32_t* seq_len, void* stream) {
    if (!problem || !bonus_target || !uniforms || !draft_token || !accepted || !out_token || !seq_tokens || !seq_len) {
        set_error("rdk_emit_sequences: null pointer");
        return RDK_ERR_INVALID_ARG;
    }
    if (problem->N < 1 || problem->batch < 1 || problem->positions < 1 || trials < 1 ||
        (problem->target_dtype != RDK_F32 && problem->target_dtype != RDK_BF16) ||
        (bonus_row_stride != 0 && bonus_row_stride < problem->N)) {
        set_error("rdk_emit_sequences: bad sizes, dtype or stride");
        return RDK_ERR_INVALID_ARG;
    }
    if (problem->N > (1 << 21)) { set_error("rdk_emit_sequences: N exceeds the supported maximum"); return RDK_ERR_UNSUPPORTED; }
    if ((long long)problem->batch * trials > 0x7fffffffLL) { set_error("rdk_emit_sequences: too many sequences"); return RDK_ERR_INVALID_ARG; }
    const int st = check_arch();
    if (st != RDK_OK) return st;
    EmitParams P;
    P.N = problem->N; P.batch = problem->batch; P.positions = problem->positions; P.trials = trials;
    P.num_tiles = (problem->N + kEmitTile - 1) / kEmitTile;
    P.bonus = bonus_target; P.bonus_stride = bonus_row_stride ? bonus_row_stride : problem->N;
    P.uniforms = uniforms; P.draft_token = draft_token; P.accepted = accepted; P.out_token = out_token;
    P.seq_tokens = seq_tokens; P.seq_len = seq_len;
    const size_t smem = (size_t)P.num_tiles * kEmitWarps * 12;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned grid = (unsigned)(problem->batch * trials);
    if (problem->target_dtype == RDK_F32) {
        RDK_CUDA(cudaFuncSetAttribute(emit_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        emit_kernel<float><<<grid, kEmitThreads, smem, s>>>(P);
    } else {
        RDK_CUDA(cudaFuncSetAttribute(emit_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        emit_kernel<__nv_bfloat16><<<grid, kEmitThreads, smem, s>>>(P);
    }
    RDK_CUDA(cudaGetLastError());
    return RDK_OK;
}
