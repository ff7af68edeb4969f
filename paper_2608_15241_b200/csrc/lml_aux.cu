// Small helper kernels: adapter packing (register_adapter), token segmentation, row gather.
#include "lml_internal.cuh"
#include "lml_ptx_sm100.cuh"

namespace lml {

// ---------------------------------------------------------------------------------------------
// register_adapter: copy A[rank][d_in] and B[d_out][rank] into the arena, zero-padded to rank 64,
// so that every kernel can read fixed-shape, 16-byte aligned rows.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_adapter_kernel(__nv_bfloat16* __restrict__ dstA,
                                                           __nv_bfloat16* __restrict__ dstB,
                                                           const __nv_bfloat16* __restrict__ A,
                                                           const __nv_bfloat16* __restrict__ B,
                                                           int rank, int d_in, int d_out)
{
    const long long nA8 = (long long)kRankPad * (d_in / 8);   // uint4 chunks of the padded A
    const long long nB = (long long)d_out * kRankPad;         // elements of the padded B
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int k8 = d_in / 8;
    for (long long i = tid; i < nA8; i += stride) {
        int j = (int)(i / k8);
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < rank) v = reinterpret_cast<const uint4*>(A)[i];   // same linear index: rows are contiguous
        reinterpret_cast<uint4*>(dstA)[i] = v;
    }
    const unsigned short* Bs = reinterpret_cast<const unsigned short*>(B);
    unsigned short* Bd = reinterpret_cast<unsigned short*>(dstB);
    for (long long i = tid; i < nB; i += stride) {
        int j = (int)(i % kRankPad);
        long long n = i / kRankPad;
        Bd[i] = (j < rank) ? Bs[n * rank + j] : (unsigned short)0;
    }
}

cudaError_t launch_pack_adapter(const Arena& ar, int slot, const void* A, const void* B, int rank,
                                int d_in, int d_out, cudaStream_t stream)
{
    __nv_bfloat16* dstA = ar.A + (size_t)slot * kRankPad * d_in;
    __nv_bfloat16* dstB = ar.B + (size_t)slot * d_out * kRankPad;
    long long work = (long long)d_out * kRankPad;
    int blocks = (int)((work + 255) / 256);
    if (blocks > 1184) blocks = 1184;
    pack_adapter_kernel<<<blocks, 256, 0, stream>>>(dstA, dstB, (const __nv_bfloat16*)A,
                                                    (const __nv_bfloat16*)B, rank, d_in, d_out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Token segmentation: stable counting sort of T tokens by slot (keys 0..max_slots-1, then -1).
// One CTA of 32 warps.  Warp w owns a contiguous range of tokens; pass 1 counts keys per warp,
// a scan turns the counts into (key-major, warp-minor) start positions, pass 2 walks the same
// range in order and places each token, using match_any to rank equal keys inside a 32-token
// chunk.  Everything is order-deterministic.
// ---------------------------------------------------------------------------------------------
constexpr int kSegWarps = 32;

// adapter id -> serving slot through the table's device map; -1 stays -1, anything else unknown is -2 (flagged)
__device__ __forceinline__ int resolve_adapter(const int32_t* __restrict__ adapter_map, int id)
{
    if (id == -1) return -1;
    if (id < 0 || id >= kMaxAdapterIds) return -2;
    const int s = __ldg(adapter_map + id);
    return s < 0 ? -2 : s;
}

__global__ void set_word_kernel(int32_t* dst, int32_t value) { *dst = value; }

cudaError_t launch_set_word(int32_t* dst, int32_t value, cudaStream_t stream)
{
    set_word_kernel<<<1, 1, 0, stream>>>(dst, value);
    return cudaGetLastError();
}

__global__ void __launch_bounds__(kSegWarps * 32) segment_tokens_kernel(
    const __grid_constant__ SlotSnapshot snap, const int32_t* __restrict__ token_slots, int T,
    int32_t* __restrict__ perm, int32_t* __restrict__ seg_offsets, int32_t* __restrict__ seg_slot_ids,
    uint32_t* __restrict__ status, const int32_t* __restrict__ adapter_map)
{
    __shared__ int hist[kSegWarps][kMaxSlots + 1];
    __shared__ int base[kMaxSlots + 2];
    const int nk = snap.max_slots + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kSegWarps * (kMaxSlots + 1); i += blockDim.x) (&hist[0][0])[i] = 0;
    ptx::grid_dependency_wait();      // launched as a programmatic dependent: whatever ran before is complete now
    ptx::grid_launch_dependents();    // the next kernel may get resident; it waits for this one the same way
    __syncthreads();

    int per = (T + kSegWarps - 1) / kSegWarps;
    per = (per + 31) & ~31;
    const int begin = min(T, warp * per);
    const int end = min(T, begin + per);
    bool bad = false;

    for (int c = begin; c < end; c += 32) {
        int i = c + lane;
        if (i < end) {
            int s = __ldg(token_slots + i);
            if (adapter_map) s = resolve_adapter(adapter_map, s);
            if (s < -1 || s >= snap.max_slots || (s >= 0 && snap.rank[s] == 0)) { bad = true; s = -1; }
            int key = s < 0 ? snap.max_slots : s;
            atomicAdd(&hist[warp][key], 1);
        }
    }
    if (bad) atomicOr(status, LML_FLAG_BAD_SLOT);
    __syncthreads();
    if ((int)threadIdx.x < nk) {
        int run = 0;
        for (int w = 0; w < kSegWarps; ++w) { int c = hist[w][threadIdx.x]; hist[w][threadIdx.x] = run; run += c; }
        base[threadIdx.x] = run;   // total of this key for now
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int k = 0; k < nk; ++k) {
            int c = base[k];
            base[k] = run;
            seg_offsets[k] = run;
            seg_slot_ids[k] = k < snap.max_slots ? k : -1;
            run += c;
        }
        seg_offsets[nk] = run;
    }
    __syncthreads();

    for (int c = begin; c < end; c += 32) {   // trip count is uniform inside a warp
        int i = c + lane;
        int key = nk;                          // sentinel for lanes past the end
        if (i < end) {
            int s = __ldg(token_slots + i);
            if (adapter_map) s = resolve_adapter(adapter_map, s);
            if (s < -1 || s >= snap.max_slots || (s >= 0 && snap.rank[s] == 0)) s = -1;
            key = s < 0 ? snap.max_slots : s;
        }
        unsigned m = __match_any_sync(0xffffffffu, key);
        int before = __popc(m & ((1u << lane) - 1u));
        int pos = 0;
        if (key < nk) {
            pos = base[key] + hist[warp][key] + before;
            perm[pos] = i;
        }
        __syncwarp();
        if (key < nk && before == 0) hist[warp][key] += __popc(m);
        __syncwarp();
    }
}

cudaError_t launch_segment_tokens(const Arena& ar, const SlotSnapshot& snap, const int32_t* token_slots,
                                  int T, int32_t* perm, int32_t* seg_offsets, int32_t* seg_slot_ids,
                                  cudaStream_t stream, bool by_adapter)
{
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3(1), dim3(kSegWarps * 32), 0, stream);
    uint32_t* status = ar.status;
    const int32_t* map = by_adapter ? ar.adapter_map : nullptr;
    return cudaLaunchKernelEx(&cfg, segment_tokens_kernel, snap, token_slots, T, perm, seg_offsets, seg_slot_ids, status, map);
}

// ---------------------------------------------------------------------------------------------
// Row gather for the perm form of the prefill call: x_grouped[p][:] = x[perm[p]][:].
// Batches usually arrive with each request's tokens together, so the grouping perm is the
// identity over long stretches.  A 128-row tile whose perm is the identity is not copied: the
// kernel marks it in tile_identity[] and the kernels that follow read (and write) those rows in
// place, with TMA, as if no perm had been given.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) gather_rows_kernel(const uint4* __restrict__ x,
                                                          const int32_t* __restrict__ perm, int T, int k8,
                                                          uint4* __restrict__ out, int32_t* __restrict__ tile_identity,
                                                          int allow_skip, uint32_t* __restrict__ status)
{
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    const int m = blockIdx.y;             // 128-row tile
    const int p0 = m * kTileM;
    const int rows = min(kTileM, T - p0);
    // every CTA of the tile takes the same decision from the same 128 perm entries
    int mine = (int)threadIdx.x < rows ? __ldg(perm + p0 + threadIdx.x) : p0 + (int)threadIdx.x;
    const int not_identity = __syncthreads_or(mine != p0 + (int)threadIdx.x);
    const bool skip = allow_skip && !not_identity;
    if (blockIdx.x == 0 && threadIdx.x == 0) tile_identity[m] = skip ? 1 : 0;
    if (skip) return;
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        const int p = p0 + r;
        int row = __ldg(perm + p);
        const bool ok = row >= 0 && row < T;
        if (!ok && threadIdx.x == 0) atomicOr(status, LML_FLAG_BAD_PERM);
        const uint4* src = x + (size_t)(ok ? row : 0) * k8;
        uint4* dst = out + (size_t)p * k8;
        for (int i = threadIdx.x; i < k8; i += blockDim.x) dst[i] = ok ? ldg_nc_v4(src + i) : make_uint4(0, 0, 0, 0);
    }
}

cudaError_t launch_gather_rows(const void* x, const int32_t* perm, int T, int d_in, void* x_grouped,
                               int32_t* tile_identity, bool allow_skip, uint32_t* status, cudaStream_t stream)
{
    dim3 grid(32, (T + kTileM - 1) / kTileM);   // 32 CTAs share a tile's 128 rows
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, grid, dim3(128), 0, stream);
    return cudaLaunchKernelEx(&cfg, gather_rows_kernel, (const uint4*)x, perm, T, d_in / 8, (uint4*)x_grouped,
                              tile_identity, allow_skip ? 1 : 0, status);
}

}  // namespace lml
