// Exact redistribution on the tensor cores (Algorithm 1 step 2):  w = q' M,  i.e.
//   w[r, j] = sum_i A[r, i] Mt[j, i]
// with A = q' (bf16, [rows, K = n], contraction index contiguous) and Mt = the transposed affinity
// matrix (bf16, [N, K]); products accumulate in fp32.
//
// One persistent CTA per SM.  A work item is a 256 x 256 tile of w: two 128 x 256 accumulators in
// tensor memory (all 512 columns), fed from a 3-stage ring of 64-wide K blocks in shared memory.
//   warp 0   : TMA producer   (cp.async.bulk.tensor, 128-byte swizzle, out-of-range rows/cols read 0)
//   warp 1   : MMA issuer     (tcgen05.mma kind::f16, one elected lane) and owner of the TMEM allocation
//   warps 2-5: epilogue       (tcgen05.ld 32 lanes x 32 columns -> fp32 stores to w)
// Items are ordered so that the row tiles of one 256-column panel of Mt run at the same time: the
// panel is fetched from HBM once and shared through L2.
// Every wait is bounded; on expiry the CTA flags RDK_ERR_TIMEOUT in the status word and winds down.
#include <cuda.h>

#include "rdk_common.cuh"

namespace rdk {

constexpr int kBM = 128;                 // rows of one MMA
constexpr int kTileM = 256;              // rows of one work item (two MMAs)
constexpr int kBN = 256;
constexpr int kBK = 64;                  // K block: 64 bf16 = 128 bytes = one swizzle row
constexpr int kStages = 3;
constexpr int kABytes = kTileM * kBK * 2;        // 32 KB
constexpr int kBBytes = kBN * kBK * 2;           // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;   // 64 KB
constexpr int kTcThreads = 192;
constexpr int kTmemCols = 512;
constexpr unsigned kTcSpin = 1u << 21;

struct TcParams {
    float* w; float* S; int rows, N, K;
    int tiles_m, tiles_n, num_kb;
    int full_items, num_items;       // items [0, full_items) are 256-row tiles, the rest 128-row halves
    int32_t* status_word;
};

// Work item -> first row, column tile and number of 128-row MMAs.  The last partial round of
// 256-row tiles is cut into 128-row halves so that it costs half a round instead of a whole one.
__device__ __forceinline__ void decode_item(const TcParams& P, int item, int& row0, int& tn, int& mt) {
    int tile, half = -1;
    if (item < P.full_items) tile = item;
    else { tile = P.full_items + ((item - P.full_items) >> 1); half = (item - P.full_items) & 1; }
    const int tm = tile % P.tiles_m;
    tn = tile / P.tiles_m;
    row0 = tm * kTileM + (half > 0 ? kBM : 0);
    const int left = P.rows - row0;
    mt = left <= 0 ? 0 : ((half < 0 && left > kBM) ? 2 : 1);
}

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Bounded wait on an mbarrier phase; false (and *abort set) when the limit is reached or another
// role has already given up.
// Called by all lanes of a warp; the answer is the same in every lane.
__device__ __forceinline__ bool tc_wait(unsigned long long* bar, uint32_t parity, volatile int* abort) {
    bool ok = false;
    for (unsigned spins = 0; spins < kTcSpin; ++spins) {
        uint32_t done;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(done) : "r"(s32(bar)), "r"(parity) : "memory");
        if (done) { ok = true; break; }
        if (*abort) break;
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) *abort = 1;
    return ok;
}

// shared-memory matrix descriptor: K-major operand, rows of 128 bytes, 128-byte swizzle, groups of
// 8 rows 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);         // start address
    d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset
    d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}

// instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = 256
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

__global__ void __launch_bounds__(kTcThreads, 1)
exact_tc_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB, const TcParams P) {
    extern __shared__ __align__(1024) unsigned char tc_smem[];
    unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) unsigned long long full_bar[kStages], empty_bar[kStages], tmem_full, tmem_empty;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < kStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(s32(&full_bar[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(s32(&empty_bar[s])));
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(s32(&tmem_full)));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" ::"r"(s32(&tmem_empty)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&tmem_base_s)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;
    const int num_items = P.num_items;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
                int row0, tn, mt;
                decode_item(P, item, row0, tn, mt);
                if (mt == 0) continue;                                        // a half tile beyond the last row
                for (int kb = 0; kb < P.num_kb; ++kb) {
                    if (!tc_wait(&empty_bar[stage], phase ^ 1u, abort)) { ok = false; break; }
                    unsigned char* sa = tiles + stage * kStageBytes;
                    if (lane == 0) {
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(&full_bar[stage])), "r"((uint32_t)kStageBytes) : "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(s32(sa)), "l"(reinterpret_cast<uint64_t>(&tmapA)), "r"(kb * kBK), "r"(row0), "r"(s32(&full_bar[stage])) : "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(s32(sa + kABytes)), "l"(reinterpret_cast<uint64_t>(&tmapB)), "r"(kb * kBK), "r"(tn * kBN), "r"(s32(&full_bar[stage])) : "memory");
                    }
                    __syncwarp();
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        {
            int stage = 0; uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
                int row0, tn, mt;
                decode_item(P, item, row0, tn, mt);                           // mt = 1: a lone 128-row remainder or half
                if (mt == 0) continue;
                if (!tc_wait(&tmem_empty, acc_phase ^ 1u, abort)) break;      // the epilogue has drained the accumulators
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kb = 0; kb < P.num_kb; ++kb) {
                    if (!tc_wait(&full_bar[stage], phase, abort)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = s32(tiles + stage * kStageBytes), b_addr = a_addr + kABytes;
                    if (lane == 0) {
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        const uint64_t bdesc = smem_desc(b_addr + k * 32);
                        for (int a = 0; a < mt; ++a) {
                            const uint64_t adesc = smem_desc(a_addr + a * (kBM * kBK * 2) + k * 32);
                            const uint32_t accum = (kb > 0 || k > 0) ? 1u : 0u;
                            asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                                         ::"r"(tmem_base + (uint32_t)(a * kBN)), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accum) : "memory");
                        }
                    }
                    // frees the stage once the MMAs above have read it
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(&empty_bar[stage])) : "memory");
                    }
                    __syncwarp();
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (lane == 0)
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(&tmem_full)) : "memory");
                __syncwarp();
                acc_phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                    // TMEM lanes 32 * quarter .. + 32 belong to this warp
        const bool vec_ok = (reinterpret_cast<uintptr_t>(P.w) & 15u) == 0 && (P.N & 3) == 0;
        uint32_t acc_phase = 0;
        for (int item = blockIdx.x; item < num_items; item += gridDim.x) {
            int row0, tn, mt;
            decode_item(P, item, row0, tn, mt);
            if (mt == 0) continue;
            if (!tc_wait(&tmem_full, acc_phase, abort)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int a = 0; a < mt; ++a) {
                const int row = row0 + a * kBM + quarter * 32 + lane;
                float* wrow = P.w + (long long)row * P.N;
                float rsum = 0.f;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * kBN + c * 32);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                        : "r"(taddr) : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int col0 = tn * kBN + c * 32;
#pragma unroll
                    for (int q = 0; q < 32; ++q) rsum += (col0 + q < P.N) ? __uint_as_float(v[q]) : 0.f;
                    if (row < P.rows) {
                        if (vec_ok && col0 + 32 <= P.N) {
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                reinterpret_cast<float4*>(wrow + col0)[q] =
                                    make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                        } else {
#pragma unroll
                            for (int q = 0; q < 32; ++q)
                                if (col0 + q < P.N) wrow[col0 + q] = __uint_as_float(v[q]);
                        }
                    }
                }
                if (P.S && row < P.rows) atomicAdd(P.S + row, rsum);           // S = sum_j w_j, one partial per tile
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(&tmem_empty)) : "memory");
            acc_phase ^= 1u;
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && abort_s && P.status_word) atomicCAS(P.status_word, 0, (int)RDK_ERR_TIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int make_map(EncodeTiledFn enc, CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_elems,
                    uint32_t box_inner, uint32_t box_outer) {
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {pitch_elems * 2};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return RDK_ERR_CUDA;
    }
    return RDK_OK;
}

int launch_exact_tc(const __nv_bfloat16* A, long long lda, const __nv_bfloat16* Mt, long long ldm, float* w_out,
                    float* S_out, int rows, int n, int N, int32_t* status_word, cudaStream_t s) {
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        RDK_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (qres != cudaDriverEntryPointSuccess || !fn) {
            set_error("rdk_redistribute_exact: the driver does not provide cuTensorMapEncodeTiled");
            return RDK_ERR_CUDA;
        }
        enc = reinterpret_cast<EncodeTiledFn>(fn);
    }
    if ((reinterpret_cast<uintptr_t>(A) & 15u) || (lda % 8) || (ldm % 8)) {
        set_error("rdk_redistribute_exact: tensor-core operands need 16-byte aligned rows");
        return RDK_ERR_INVALID_ARG;
    }
    CUtensorMap mapA, mapB;
    int st = make_map(enc, &mapA, A, (uint64_t)n, (uint64_t)rows, (uint64_t)lda, kBK, kTileM);
    if (st != RDK_OK) return st;
    st = make_map(enc, &mapB, Mt, (uint64_t)n, (uint64_t)N, (uint64_t)ldm, kBK, kBN);
    if (st != RDK_OK) return st;
    TcParams P;
    P.w = w_out; P.S = S_out; P.rows = rows; P.N = N; P.K = n;
    P.tiles_m = (rows + kTileM - 1) / kTileM;
    P.tiles_n = (N + kBN - 1) / kBN;
    P.num_kb = (n + kBK - 1) / kBK;
    P.status_word = status_word;
    int dev = 0, sms = 0;
    RDK_CUDA(cudaGetDevice(&dev));
    RDK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long tiles = (long long)P.tiles_m * P.tiles_n;
    if (tiles > 0x3fffffffLL) { set_error("rdk_redistribute_exact: too many output tiles"); return RDK_ERR_UNSUPPORTED; }
    const int grid = (int)(tiles < sms ? tiles : sms);
    const int rest = (int)(tiles % grid);
    const bool split = rest > 0 && 2 * rest <= grid && tiles > grid;      // cut the last partial round into halves
    P.full_items = split ? (int)(tiles - rest) : (int)tiles;
    P.num_items = split ? (int)(tiles + rest) : (int)tiles;
    if (S_out) RDK_CUDA(cudaMemsetAsync(S_out, 0, (size_t)rows * sizeof(float), s));
    const size_t smem = (size_t)kStages * kStageBytes + 1024;
    RDK_CUDA(cudaFuncSetAttribute(exact_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    exact_tc_kernel<<<grid, kTcThreads, smem, s>>>(mapA, mapB, P);
    RDK_CUDA(cudaGetLastError());
    return RDK_OK;
}

}  // namespace rdk
