// Kept-id index: membership bitmask over the target vocabulary, per-word rank counts and the
// rank -> drafter-index table.  The intersection I = T n D of Sec. 2 is "ids inside [0, N)";
// everything else is the out-of-vocabulary set F that Token-Level Intersection drops.
#include <mutex>
#include <unordered_map>

#include "rdk_common.cuh"

namespace rdk {

static std::mutex g_order_mu;
struct IndexNote { int N, n; bool ascending_valid; };
static std::unordered_map<const void*, IndexNote>& order_map() {
    static std::unordered_map<const void*, IndexNote> m;
    return m;
}
void note_index_order(const void* kept_index, int N, int n, bool ascending_valid) {
    std::lock_guard<std::mutex> lk(g_order_mu);
    order_map()[kept_index] = IndexNote{N, n, ascending_valid};
}
int index_order(const void* kept_index, int N, int n) {
    std::lock_guard<std::mutex> lk(g_order_mu);
    auto it = order_map().find(kept_index);
    if (it == order_map().end() || it->second.N != N || it->second.n != n) return -1;
    return it->second.ascending_valid ? 1 : 0;
}

__global__ void idx_clear_kernel(int32_t* header, uint32_t* mask, int32_t* slot, int words, int N, int n) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    const int stride = gridDim.x * blockDim.x;
    for (int w = g; w < words; w += stride) mask[w] = 0u;
    for (int i = g; i < n; i += stride) slot[i] = -1;
    if (g == 0) {
        for (int k = 0; k < 64; ++k) header[k] = 0;
        header[kHdrN] = N;
        header[kHdrn] = n;
        header[kHdrIdentity] = 1;
    }
}

__global__ void idx_mark_kernel(const int32_t* __restrict__ ids, int32_t* ids_copy, int32_t* header,
                                uint32_t* mask, int N, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int id = ids[i];
    ids_copy[i] = id;
    if (id >= 0 && id < N) {
        const uint32_t bit = 1u << (id & 31);
        const uint32_t old = atomicOr(&mask[id >> 5], bit);
        if (old & bit) atomicExch(&header[kHdrDup], 1);
        atomicAdd(&header[kHdrValid], 1);
    }
}

// One CTA: exclusive prefix sum of the per-word popcounts.
__global__ void idx_rank_kernel(const uint32_t* __restrict__ mask, int32_t* rank, int words) {
    __shared__ int warp_tot[32];
    __shared__ int carry;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int w0 = 0; w0 < words; w0 += blockDim.x) {
        const int w = w0 + threadIdx.x;
        const int c = (w < words) ? __popc(mask[w]) : 0;
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        int before = carry;
        for (int k = 0; k < wid; ++k) before += warp_tot[k];
        if (w < words) rank[w] = before + incl - c;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = carry;
            for (int k = 0; k < nw; ++k) t += warp_tot[k];
            carry = t;
        }
        __syncthreads();
    }
}

__global__ void idx_slot_kernel(const int32_t* __restrict__ ids, const uint32_t* __restrict__ mask,
                                const int32_t* __restrict__ rank, int32_t* slot, int32_t* header,
                                int N, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int id = ids[i];
    if (id < 0 || id >= N) {
        atomicExch(&header[kHdrIdentity], 0);   // a dropped entry shifts every later rank
        return;
    }
    const uint32_t word = mask[id >> 5];
    const int r = rank[id >> 5] + __popc(word & ((1u << (id & 31)) - 1u));
    slot[r] = i;                                 // duplicates (rejected by the host) would collide here
    if (r != i) atomicExch(&header[kHdrIdentity], 0);
}

// Tables of the streaming kernels for one target element size (ascending valid ids only: rank =
// drafter index).  Segment s covers tokens [s Lw, (s + 1) Lw); its kept tokens are the drafter
// indices [r_lo, r_hi).  The kernels read drafter values in aligned pairs, so the segment's slot
// grid starts at the even index r0 <= r_lo (slot 0 is a "dummy" of the previous segment when r_lo is
// odd) and is padded to a multiple of 64 slots.
// One CTA of kStreamMaxSeg threads: per-segment descriptors {r0, slots in use, table start, dummy}.
__global__ void idx_segdesc_kernel(const uint32_t* __restrict__ mask, const int32_t* __restrict__ rank,
                                   int4* segdesc, int N, int n, int Lw) {
    __shared__ int padded[kStreamMaxSeg];
    const int s = threadIdx.x;
    auto rank_at = [&](long long j) -> int {
        if (j >= N) return n;
        const uint32_t word = mask[j >> 5];
        return rank[j >> 5] + __popc(word & ((1u << (j & 31)) - 1u));
    };
    const long long j0 = (long long)s * Lw;
    const int r_lo = rank_at(j0), r_hi = rank_at(j0 + Lw);
    const int dummy = r_lo & 1, r0 = r_lo - dummy, kcp = r_hi - r0;
    padded[s] = (kcp + 63) & ~63;
    __syncthreads();
    int start = 0;
    for (int k = 0; k < s; ++k) start += padded[k];
    segdesc[s] = make_int4(r0, kcp, start, dummy);
}

// One CTA per segment: byte offset, inside the slice of the CTA that owns the segment, of the
// target logit of every slot; slots without a kept token of the segment point at the spare
// element behind the slice, which the kernels keep at weight zero.
__global__ void idx_goff_kernel(const int32_t* __restrict__ ids, const int4* __restrict__ segdesc,
                                uint16_t* goff, int N, int Lw, int es) {
    const int s = blockIdx.x;
    const int4 d = segdesc[s];
    const int padded = (d.y + 63) & ~63;
    const long long j0 = (long long)s * Lw;
    const int w = s % kStreamWarps;
    const unsigned spare = (unsigned)kStreamWarps * (unsigned)Lw * (unsigned)es;
    for (int il = threadIdx.x; il < padded; il += blockDim.x) {
        unsigned o = spare;
        if (il < d.y && !(d.w && il == 0))
            o = ((unsigned)w * (unsigned)Lw + (unsigned)(ids[d.x + il] - j0)) * (unsigned)es;
        goff[d.z + il] = (uint16_t)o;
    }
}

__global__ void idx_seal_kernel(int32_t* header, int plan) {
    header[kHdrPlan] = plan;
    header[kHdrMagic] = kIdxMagic;
}

}  // namespace rdk

using namespace rdk;

extern "C" size_t rdk_kept_index_bytes(int32_t N, int32_t n) {
    if (N < 1 || n < 1) return 0;
    return idx_bytes(N, n);
}

extern "C" int rdk_prepare_ids(const int32_t* kept_ids, int32_t n, int32_t N, void* kept_index,
                               size_t kept_index_bytes, int* n_valid_host, void* stream) {
    if (!kept_ids || !kept_index || N < 1 || n < 1) {
        set_error("rdk_prepare_ids: null pointer or non-positive size (N=%d n=%d)", N, n);
        return RDK_ERR_INVALID_ARG;
    }
    if ((reinterpret_cast<uintptr_t>(kept_index) & 255u) != 0) {
        set_error("rdk_prepare_ids: kept_index must be 256-byte aligned");
        return RDK_ERR_INVALID_ARG;
    }
    if (kept_index_bytes < idx_bytes(N, n)) {
        set_error("rdk_prepare_ids: buffer has %zu bytes, %zu needed", kept_index_bytes, idx_bytes(N, n));
        return RDK_ERR_WORKSPACE_TOO_SMALL;
    }
    const int st = check_arch();
    if (st != RDK_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    KeptIndexView v = make_view(kept_index, N, n);
    int32_t* header = const_cast<int32_t*>(v.header);
    uint32_t* mask = const_cast<uint32_t*>(v.mask);
    int32_t* rank = const_cast<int32_t*>(v.rank);
    int32_t* slot = const_cast<int32_t*>(v.slot);
    int32_t* ids = const_cast<int32_t*>(v.ids);
    const int tb = 256;
    const int work = v.words > n ? v.words : n;
    int blocks = (work + tb - 1) / tb;
    if (blocks > 1184) blocks = 1184;
    idx_clear_kernel<<<blocks, tb, 0, s>>>(header, mask, slot, v.words, N, n);
    idx_mark_kernel<<<(n + tb - 1) / tb, tb, 0, s>>>(kept_ids, ids, header, mask, N, n);
    idx_rank_kernel<<<1, 1024, 0, s>>>(mask, rank, v.words);
    idx_slot_kernel<<<(n + tb - 1) / tb, tb, 0, s>>>(ids, mask, rank, slot, header, N, n);
    RDK_CUDA(cudaGetLastError());
    int32_t host_hdr[8] = {0};
    RDK_CUDA(cudaMemcpyAsync(host_hdr, header, sizeof(host_hdr), cudaMemcpyDeviceToHost, s));
    RDK_CUDA(cudaStreamSynchronize(s));
    if (n_valid_host) *n_valid_host = host_hdr[kHdrValid];
    note_index_order(kept_index, N, n, host_hdr[kHdrIdentity] != 0 && host_hdr[kHdrValid] == n);
    if (host_hdr[kHdrDup]) {
        set_error("rdk_prepare_ids: two drafter indices map to the same target token");
        return RDK_ERR_BAD_IDS;
    }
    if (host_hdr[kHdrValid] == 0) {
        set_error("rdk_prepare_ids: no kept id lies inside the target vocabulary [0, %d)", N);
        return RDK_ERR_EMPTY_INTERSECTION;
    }
    // ascending valid ids: the streaming kernels' tables, for 2-byte and 4-byte target logits
    int plan = 0;
    if (host_hdr[kHdrIdentity] != 0 && host_hdr[kHdrValid] == n) {
        for (int k = 0; k < 2; ++k) {
            StreamSegs g;
            const int es = k == 0 ? 2 : 4;
            if (!stream_segments(N, (size_t)es, g)) continue;
            int4* sd = const_cast<int4*>(v.segdesc[k]);
            idx_segdesc_kernel<<<1, kStreamMaxSeg, 0, s>>>(mask, rank, sd, N, n, g.Lw);
            idx_goff_kernel<<<kStreamMaxSeg, 128, 0, s>>>(ids, sd, const_cast<uint16_t*>(v.goff[k]), N, g.Lw, es);
            plan |= 1 << k;
        }
    }
    idx_seal_kernel<<<1, 1, 0, s>>>(header, plan);
    RDK_CUDA(cudaGetLastError());
    RDK_CUDA(cudaStreamSynchronize(s));
    return RDK_OK;
}
