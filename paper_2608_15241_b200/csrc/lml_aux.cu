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
                                                           __nv_bfloat16* __restrict__ dstBc,
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
    if (rank <= kRankCompact) {   // the compact copy: [d_out][kRankCompact]
        unsigned short* Bcd = reinterpret_cast<unsigned short*>(dstBc);
        for (long long i = tid; i < (long long)d_out * kRankCompact; i += stride) {
            const int j = (int)(i % kRankCompact);
            const long long n = i / kRankCompact;
            Bcd[i] = (j < rank) ? Bs[n * rank + j] : (unsigned short)0;
        }
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
    __nv_bfloat16* dstBc = ar.Bc + (size_t)slot * d_out * kRankCompact;
    pack_adapter_kernel<<<blocks, 256, 0, stream>>>(dstA, dstB, dstBc, (const __nv_bfloat16*)A,
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
constexpr int kSegKeyCache = 16384;   // tokens whose keys are kept in shared memory between the two passes

__global__ void set_word_kernel(int32_t* dst, int32_t value) { *dst = value; }
__global__ void clear_word_if_kernel(int32_t* dst, int32_t expected) { if (*dst == expected) *dst = -1; }

cudaError_t launch_clear_word_if(int32_t* dst, int32_t expected, cudaStream_t stream)
{
    clear_word_if_kernel<<<1, 1, 0, stream>>>(dst, expected);
    return cudaGetLastError();
}

cudaError_t launch_set_word(int32_t* dst, int32_t value, cudaStream_t stream)
{
    set_word_kernel<<<1, 1, 0, stream>>>(dst, value);
    return cudaGetLastError();
}

// Host-buffer form of a decode call whose host buffers are pinned: one kernel pulls the inputs out of
// host memory (16-byte loads for x, all in flight at once: one trip over the host link instead of a DMA
// copy per array) into the device staging that the decode kernel reads.
__global__ void __launch_bounds__(256) stage_host_inputs_kernel(
    const uint4* __restrict__ x_host, uint4* __restrict__ x_dev, int x_chunks, const int32_t* __restrict__ so_host,
    int32_t* __restrict__ so_dev, int n_so, const int32_t* __restrict__ ids_host, int32_t* __restrict__ ids_dev, int n_ids,
    const int32_t* __restrict__ perm_host, int32_t* __restrict__ perm_dev, int n_perm)
{
    ptx::grid_dependency_wait();   // the call before may still read the staging
    ptx::grid_launch_dependents();
    const int i = blockIdx.x * blockDim.x + threadIdx.x, n = gridDim.x * blockDim.x;
    for (int c = i; c < x_chunks; c += n) x_dev[c] = x_host[c];
    for (int c = i; c < n_so; c += n) so_dev[c] = so_host[c];
    for (int c = i; c < n_ids; c += n) ids_dev[c] = ids_host[c];
    for (int c = i; c < n_perm; c += n) perm_dev[c] = perm_host[c];
}

cudaError_t launch_stage_host_inputs(const void* x_host, void* x_dev, size_t x_bytes, const int32_t* so_host, int32_t* so_dev,
                                     int n_so, const int32_t* ids_host, int32_t* ids_dev, int n_ids,
                                     const int32_t* perm_host, int32_t* perm_dev, int n_perm, cudaStream_t stream)
{
    const int chunks = (int)(x_bytes / 16);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3((unsigned)((chunks + 255) / 256 < 1 ? 1 : (chunks + 255) / 256)), dim3(256), 0, stream);
    return cudaLaunchKernelEx(&cfg, stage_host_inputs_kernel, (const uint4*)x_host, (uint4*)x_dev, chunks, so_host, so_dev,
                              n_so, ids_host, ids_dev, n_ids, perm_host, perm_dev, n_perm);
}

// Host-buffer form of large calls, done chunk by chunk: the segment arrays of chunk c (rows [c * rows,
// (c + 1) * rows) of the call), offsets relative to the chunk and clipped to it.  Malformed offsets are
// detected on the whole call and poison every chunk's array, so that every chunk falls back to the base
// output, as the unchunked call does.
__global__ void __launch_bounds__(256) clip_segments_kernel(const int32_t* __restrict__ seg_offsets,
                                                            const int32_t* __restrict__ slot_ids, int G, int T, int rows,
                                                            int32_t* __restrict__ out, int stride)
{
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    const int c = blockIdx.x, r0 = c * rows, Tc = min(rows, T - r0);
    int32_t* so = out + (size_t)c * stride;
    int32_t* ids = so + G + 1;
    int bad = 0;
    for (int g = threadIdx.x; g < G; g += blockDim.x) {
        const int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1);
        if (s1 < s0 || s0 < 0 || s1 > T) bad = 1;
    }
    if (threadIdx.x == 0 && (__ldg(seg_offsets) != 0 || __ldg(seg_offsets + G) != T)) bad = 1;
    bad = __syncthreads_or(bad);
    for (int g = threadIdx.x; g <= G; g += blockDim.x) {
        const int v = min(max(__ldg(seg_offsets + g) - r0, 0), Tc);
        so[g] = bad ? (g == 0 ? 1 : 0) : v;   // (an array that starts at 1 is malformed for every chunk)
        if (g < G) ids[g] = __ldg(slot_ids + g);
    }
}

cudaError_t launch_clip_segments(const int32_t* seg_offsets, const int32_t* slot_ids, int G, int T, int rows, int chunks,
                                 int32_t* out, int stride, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3((unsigned)chunks), dim3(256), 0, stream);
    return cudaLaunchKernelEx(&cfg, clip_segments_kernel, seg_offsets, slot_ids, G, T, rows, out, stride);
}

__global__ void __launch_bounds__(kSegWarps * 32) segment_tokens_kernel(
    const __grid_constant__ SlotSnapshot snap, const int32_t* __restrict__ token_slots, int T,
    int32_t* __restrict__ perm, int32_t* __restrict__ seg_offsets, int32_t* __restrict__ seg_slot_ids,
    uint32_t* __restrict__ status, const int32_t* __restrict__ adapter_map)
{
    __shared__ int hist[kSegWarps][kMaxSlots + 1];
    __shared__ int base[kMaxSlots + 2];
    __shared__ uint8_t keys_s[kSegKeyCache];
    const int nk = snap.max_slots + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kSegWarps * (kMaxSlots + 1); i += blockDim.x) (&hist[0][0])[i] = 0;
    ptx::grid_dependency_wait();      // launched as a programmatic dependent: whatever ran before is complete now
    ptx::grid_launch_dependents();    // the next kernel may get resident; it waits for this one the same way
    // Up to kSegKeyCache tokens: every key is fetched once, all loads in flight together (one trip to memory instead of
    // one per 32 tokens of a warp's range and pass), and both passes read shared memory.  0xff marks an id that names
    // no live slot (it counts as "none" and raises the flag).
    const bool cached = T <= kSegKeyCache;
    if (cached) {
        for (int i = threadIdx.x; i < T; i += blockDim.x) {
            int s = __ldg(token_slots + i);
            if (adapter_map) s = resolve_adapter(snap, adapter_map, s);
            const bool bad_id = s < -1 || s >= snap.max_slots || (s >= 0 && snap.rank[s] == 0);
            keys_s[i] = bad_id ? (uint8_t)0xff : (uint8_t)(s < 0 ? snap.max_slots : s);
        }
    }
    __syncthreads();

    int per = (T + kSegWarps - 1) / kSegWarps;
    per = (per + 31) & ~31;
    const int begin = min(T, warp * per);
    const int end = min(T, begin + per);
    bool bad = false;

    for (int c = begin; c < end; c += 32) {
        int i = c + lane;
        if (i < end) {
            int key;
            if (cached) {
                key = keys_s[i];
                if (key == 0xff) { bad = true; key = snap.max_slots; }
            } else {
                int s = __ldg(token_slots + i);
                if (adapter_map) s = resolve_adapter(snap, adapter_map, s);
                if (s < -1 || s >= snap.max_slots || (s >= 0 && snap.rank[s] == 0)) { bad = true; s = -1; }
                key = s < 0 ? snap.max_slots : s;
            }
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
            if (cached) {
                key = keys_s[i] == 0xff ? snap.max_slots : (int)keys_s[i];
            } else {
                int s = __ldg(token_slots + i);
                if (adapter_map) s = resolve_adapter(snap, adapter_map, s);
                if (s < -1 || s >= snap.max_slots || (s >= 0 && snap.rank[s] == 0)) s = -1;
                key = s < 0 ? snap.max_slots : s;
            }
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
// Token-form calls of a row tile or two (T <= 128 or 256) that are too long for the decode kernel: binding and shrink in
// one launch, with no grouping and no row copy.  The GEMM adds, per LoRA piece of a row tile, the product of a whole
// 128 x 64 block of u with the slot's B; which rows of the block are non-zero is the block's own business.  So the
// tokens stay in their order: the distinct live slots of a tile's tokens, in ascending order, become the tile's
// "segments" (the k-th is given the row range [128 m + k, 128 m + k + 1), the tile's last one the rest of the tile:
// ranges that lie in their tile and satisfy the layer's checks; the GEMM only asks which tile a range meets; a tile
// without any slot gets one segment without a slot), numbered through the tiles, and the block of segment g of tile m,
// block m + g as on the grouped path, holds scale * x_t . A_slot^T in the tile's rows t that are bound to that slot and
// zeros everywhere else.  (The kernel serves up to eight tiles; beyond two the GEMM's extra pieces, one per slot and
// tile, cost more than grouping the rows: 54.9 against 48.2 us at 1024 tokens on 4096 x 4096.)
// One CTA per row: it works out the slot sets of its tile and of the tiles before it, computes its row's dot
// products (up to sixteen columns j at a time, one or two warps per column, each on its part of the row; the row of x
// in shared memory when it fits) and writes its row of every block.  The GEMM that follows (216 KB of shared memory and
// 18K registers per CTA) gets resident beside this kernel's CTAs, and starts on its base k-blocks, only where they leave
// it room: 512 threads of at most 64 registers and a row of x of at most 8 KB do (d_in <= 4096); a wider row does not
// fit beside the GEMM anyway, and 1024 threads finish it sooner.  Measured, us per call at 128 tokens on 4096 x 4096 /
// 11008 x 4096 / 4096 x 11008: 256 threads 23.9 / 32.1 / 47.7, 512 threads 21.2 / 32.2 / 40.2, 1024 threads 24.4 / 39.6 /
// 37.8; 512 threads with sixteen loads in flight per lane (128 registers) 25.2 / 39.9 / 40.8.  (A small persistent grid
// on the SMs that the GEMM leaves free was measured too: beside the GEMM's stream every dependent load takes
// microseconds, 37 against 21 us per call.)
constexpr int kBindMaxSmemCols = 20480;   // a row of x up to this width is staged in shared memory (40 KB)
constexpr int kBindMaxTiles = 8;          // row tiles of a call at most

template <int kThreads>
__global__ void __launch_bounds__(kThreads) bind_shrink_tile_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaA,
    const int32_t* __restrict__ token_slots, int T, int K, const __nv_bfloat16* __restrict__ x,
    int32_t* __restrict__ seg_offsets, int32_t* __restrict__ seg_slot_ids, int G, PlanWord* __restrict__ plan,
    __nv_bfloat16* __restrict__ u_blocks, uint32_t* __restrict__ status, const int32_t* __restrict__ adapter_map, int in_smem)
{
    constexpr int kWarps = kThreads / 32;
    constexpr int kCols = kWarps < 16 ? kWarps : 16;   // columns worked on side by side
    constexpr int kParts = kWarps / kCols;             // warps per column, each on its part of the row
    extern __shared__ uint4 bind_x_s[];
    __shared__ unsigned mask_s[kBindMaxTiles][2];
    __shared__ int my_slot_s, bad_s;
    __shared__ float dots_s[kRankPad];
    __shared__ float part_s[kParts][kRankPad];
    const int row = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = row / kTileM, r_in_tile = row % kTileM, num_m = (T + kTileM - 1) / kTileM;
    if (tid < 2 * kBindMaxTiles) (&mask_s[0][0])[tid] = 0u;
    if (tid == 0) { my_slot_s = -1; bad_s = 0; }
    ptx::grid_dependency_wait();      // launched as a programmatic dependent: whatever ran before is complete now
    ptx::grid_launch_dependents();    // the GEMM may get resident where there is room; it waits for this grid before its pieces
    __syncthreads();
    const int nch = K / 8;
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * K);
    if (row < T && in_smem)   // (does not depend on the binding: goes out with the ids)
        for (int c = tid; c < nch; c += kThreads) bind_x_s[c] = __ldg(xr + c);
    // the slot sets of this row's tile and of the tiles before it (their sizes place this tile's segments and blocks)
    const bool closes = tile == num_m - 1 && r_in_tile == 0;   // the CTA that also closes the segment arrays
    const int ids_end = min(T, (tile + 1) * kTileM);
    for (int i = tid; i < ids_end; i += kThreads) {
        int s = __ldg(token_slots + i);
        if (adapter_map) s = resolve_adapter(snap, adapter_map, s);
        const bool bad_id = s < -1 || s >= snap.max_slots || (s >= 0 && snap.rank[s] == 0);
        if (bad_id) { bad_s = 1; s = -1; }
        if (s >= 0) atomicOr(&mask_s[i / kTileM][s >> 5], 1u << (s & 31));
        if (i == row) my_slot_s = s;
    }
    __syncthreads();
    // A tile's segments: one per distinct live slot of the tile, in ascending order; a tile without any gets one
    // segment without a slot, so that every tile's rows belong to segments of its own.
    auto tile_mask = [&](int m) { return (unsigned long long)mask_s[m][0] | ((unsigned long long)mask_s[m][1] << 32); };
    int base = 0;   // segments of the tiles before this one
    for (int m = 0; m < tile; ++m) base += max(1, __popcll(tile_mask(m)));
    const unsigned long long mask = tile_mask(tile);
    const int Gp = __popcll(mask);
    if (r_in_tile == 0) {
        if (tid == 0 && bad_s && closes) atomicOr(status, LML_FLAG_BAD_SLOT);   // (this CTA has seen every id)
        const int nseg = max(1, Gp);
        for (int k = tid; k < nseg; k += kThreads) {
            int slot = -1;
            if (k < Gp) {   // the k-th live slot of the tile
                unsigned long long mm = mask;
                for (int q = 0; q < k; ++q) mm &= mm - 1ull;
                slot = __ffsll((long long)mm) - 1;
            }
            seg_offsets[base + k] = tile * kTileM + k;
            seg_slot_ids[base + k] = slot;
        }
        if (closes) {
            for (int g = base + nseg + tid; g <= G; g += kThreads) {
                seg_offsets[g] = T;
                if (g < G) seg_slot_ids[g] = -1;
            }
            if (tid == 0) plan->lora_ok = 1;
        }
    }
    const int my_slot = row < T ? my_slot_s : -1;
    const int g_mine = my_slot >= 0 ? __popcll(mask & ((1ull << my_slot) - 1ull)) : -1;
    const int rank = my_slot >= 0 ? (int)snap.rank[my_slot] : 0;
    // this row's dot products: the warps w, w + kCols, ... take the columns j = w, w + kCols, ..., each its part of the
    // row; a lane sums the 8-element chunks lane, lane + 32, ... of the part in order, the warp adds its lanes up with
    // the butterfly, and the parts are added in a fixed order
    const int part = (nch + kParts - 1) / kParts;
    const int h = warp / kCols, c_begin = min(nch, h * part), c_end = min(nch, c_begin + part);
    for (int j = warp % kCols; j < rank; j += kCols) {
        const uint4* ar = reinterpret_cast<const uint4*>(arenaA + ((size_t)my_slot * kRankPad + j) * K);
        float acc = 0.f;
        for (int c0 = c_begin + lane; c0 < c_end; c0 += 32 * 8) {
            uint4 av[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int c = c0 + 32 * i;
                av[i] = c < c_end ? __ldg(ar + c) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int c = c0 + 32 * i;
                if (c < c_end) {
                    const uint4 xv = in_smem ? bind_x_s[c] : __ldg(xr + c);
                    float p = 0.f;
                    p = fmaf(bf16_lo(xv.x), bf16_lo(av[i].x), p); p = fmaf(bf16_hi(xv.x), bf16_hi(av[i].x), p);
                    p = fmaf(bf16_lo(xv.y), bf16_lo(av[i].y), p); p = fmaf(bf16_hi(xv.y), bf16_hi(av[i].y), p);
                    p = fmaf(bf16_lo(xv.z), bf16_lo(av[i].z), p); p = fmaf(bf16_hi(xv.z), bf16_hi(av[i].z), p);
                    p = fmaf(bf16_lo(xv.w), bf16_lo(av[i].w), p); p = fmaf(bf16_hi(xv.w), bf16_hi(av[i].w), p);
                    acc += p;
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) part_s[h][j] = acc;
    }
    __syncthreads();
    if (tid < kRankPad) {
        float v = 0.f;
        if (tid < rank) {
#pragma unroll
            for (int q = 0; q < kParts; ++q) v += part_s[q][tid];
            v *= snap.scale[my_slot];
        }
        dots_s[tid] = v;
    }
    __syncthreads();
    // this row of every block: the dot products in its own block, zeros in the others (pairs of columns per thread)
    for (int i = tid; i < Gp * (kRankPad / 2); i += kThreads) {
        const int g = i / (kRankPad / 2), c2 = i % (kRankPad / 2);
        __nv_bfloat162 v = __floats2bfloat162_rn(0.f, 0.f);
        if (g == g_mine) v = __floats2bfloat162_rn(dots_s[2 * c2], dots_s[2 * c2 + 1]);
        reinterpret_cast<__nv_bfloat162*>(u_blocks + ((size_t)(tile + base + g) * kTileM + r_in_tile) * kRankPad)[c2] = v;
    }
}

cudaError_t launch_bind_shrink_tile(const Arena& ar, const SlotSnapshot& snap, const int32_t* token_slots, int T, int d_in,
                                    const void* x, int32_t* seg_offsets, int32_t* seg_slot_ids, int G, PlanWord* plan,
                                    void* u_blocks, int threads, cudaStream_t stream, bool by_adapter)
{
    const int in_smem = d_in <= kBindMaxSmemCols ? 1 : 0;   // (reading x through L1 instead was measured: 2 - 7 us slower per call)
    const size_t smem = in_smem ? (size_t)d_in * 2 : 0;   // (at most 40 KB: no opt-in needed)
    auto launch = [&](auto kernel, int nthreads) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        pdl_config(cfg, attr, dim3((unsigned)(((T + kTileM - 1) / kTileM) * kTileM)), dim3((unsigned)nthreads), smem, stream);
        return cudaLaunchKernelEx(&cfg, kernel, snap, (const __nv_bfloat16*)ar.A, token_slots, T, d_in,
                                  (const __nv_bfloat16*)x, seg_offsets, seg_slot_ids, G, plan, (__nv_bfloat16*)u_blocks, ar.status,
                                  by_adapter ? (const int32_t*)ar.adapter_map : (const int32_t*)nullptr, in_smem);
    };
    if (threads >= 1024) return launch(bind_shrink_tile_kernel<1024>, 1024);
    if (threads >= 512) return launch(bind_shrink_tile_kernel<512>, 512);
    return launch(bind_shrink_tile_kernel<256>, 256);
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

// ---------------------------------------------------------------------------------------------
// Transposed registration for the backward pass: the gradient with respect to x of the layer
// (d_in = K, d_out = N, adapter A [r][K], B [N][r]) is the layer itself on the transposed problem
// (d_in = N, d_out = K, base weight W0^T, adapter A' = B^T [r][N], B' = A^T [K][r]).  This kernel
// packs (A', B') into the arena of the transposed table straight from the caller's A and B.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_adapter_transposed_kernel(__nv_bfloat16* __restrict__ dstA,
                                                                      __nv_bfloat16* __restrict__ dstB,
                                                                      __nv_bfloat16* __restrict__ dstBc,
                                                                      const __nv_bfloat16* __restrict__ A,
                                                                      const __nv_bfloat16* __restrict__ B,
                                                                      int rank, int K, int N)
{
    const unsigned short* As = reinterpret_cast<const unsigned short*>(A);
    const unsigned short* Bs = reinterpret_cast<const unsigned short*>(B);
    unsigned short* Ad = reinterpret_cast<unsigned short*>(dstA);   // [64][N]: A'[j][n] = B[n][j]
    unsigned short* Bd = reinterpret_cast<unsigned short*>(dstB);   // [K][64]: B'[k][j] = A[j][k]
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (long long i = tid; i < (long long)kRankPad * N; i += stride) {
        const int j = (int)(i / N);
        const long long n = i % N;
        Ad[i] = j < rank ? Bs[n * rank + j] : (unsigned short)0;
    }
    for (long long i = tid; i < (long long)K * kRankPad; i += stride) {
        const int j = (int)(i % kRankPad);
        const long long k = i / kRankPad;
        Bd[i] = j < rank ? As[(long long)j * K + k] : (unsigned short)0;
    }
    if (rank <= kRankCompact) {   // the compact copy of B': [K][kRankCompact]
        unsigned short* Bcd = reinterpret_cast<unsigned short*>(dstBc);
        for (long long i = tid; i < (long long)K * kRankCompact; i += stride) {
            const int j = (int)(i % kRankCompact);
            const long long k = i / kRankCompact;
            Bcd[i] = j < rank ? As[(long long)j * K + k] : (unsigned short)0;
        }
    }
}

cudaError_t launch_pack_adapter_transposed(const Arena& arT, int slot, const void* A, const void* B, int rank,
                                           int K, int N, cudaStream_t stream)
{
    __nv_bfloat16* dstA = arT.A + (size_t)slot * kRankPad * N;   // the transposed table has d_in = N ...
    __nv_bfloat16* dstB = arT.B + (size_t)slot * K * kRankPad;   // ... and d_out = K
    long long work = (long long)(K > N ? K : N) * kRankPad;
    int blocks = (int)((work + 255) / 256);
    if (blocks > 1184) blocks = 1184;
    __nv_bfloat16* dstBc = arT.Bc + (size_t)slot * K * kRankCompact;
    pack_adapter_transposed_kernel<<<blocks, 256, 0, stream>>>(dstA, dstB, dstBc, (const __nv_bfloat16*)A,
                                                               (const __nv_bfloat16*)B, rank, K, N);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Adapter gradients: out_s += P_s^T . Q_s over the tokens bound to slot s, where P holds one
// 64-wide row per position (the piece blocks a shrink pass wrote: scale.(dy.B) for dA, scale.(x.A^T)
// for dB) and Q is x (for dA, C = d_in) or dy (for dB, C = d_out).  One CTA of eight warps per
// (128 columns, slot), two CTAs to an SM; the contraction over positions runs on mma.sync (see the
// kernel), the slot's positions are walked in order and the sums stay in registers, so the result does
// not depend on scheduling.  fp32 accumulation, added onto what out holds.
// mode 0: out[slot][j][c] (dA);  mode 1: out[slot][c][j] (dB).
// ---------------------------------------------------------------------------------------------
constexpr int kGradCols = 128;                                  // columns of Q (and of the output) per CTA: two CTAs fit on an SM
constexpr int kGradQPitch = kGradCols * 2 + 16;                 // bytes per row of the staged Q tile (16 more: no bank conflicts in ldmatrix)
constexpr int kGradPPitch = kRankPad * 2 + 16;                  // bytes per row of the staged piece block
constexpr int kGradQBytes = kTileM * kGradQPitch;
constexpr int kGradPBytes = kTileM * kGradPPitch;
constexpr int kGradSmemBytes = 2 * (kGradQBytes + kGradPBytes); // two work items in flight

__device__ __forceinline__ void grad_cp_async_16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

// out_s (64 x C) += P_s^T (64 x positions) . Q_s (positions x C) on mma.sync m16n8k16: the contraction
// runs over positions, 16 at a time.  P is staged as [position][j] and Q as [position][column], so both
// operands are read with ldmatrix .trans.  Warp w owns columns 16w .. 16w+15 (two 8-wide tiles) and all
// 16-row groups of j that the slot's rank needs.
// One launch does both gradients side by side: blockIdx.z = 0 takes the first set of arguments, 1 the second.
struct GradJob {
    const __nv_bfloat16* pieces;
    const __nv_bfloat16* Q;
    float* out;
    int C, mode;
};
__global__ void __launch_bounds__(256, 2) weight_grad_kernel(const __grid_constant__ SlotSnapshot snap, const GradJob job0,
                                                          const GradJob job1, int T,
                                                          const int32_t* __restrict__ seg_offsets,
                                                          const int32_t* __restrict__ slot_ids, int G)
{
    extern __shared__ __align__(16) unsigned char grad_smem[];
    ptx::grid_dependency_wait();     // the shrink passes before this kernel are complete now
    ptx::grid_launch_dependents();
    const GradJob& job = blockIdx.z == 0 ? job0 : job1;
    const __nv_bfloat16* __restrict__ pieces = job.pieces;
    const __nv_bfloat16* __restrict__ Q = job.Q;
    float* __restrict__ out = job.out;
    const int C = job.C, mode = job.mode;
    if ((int)blockIdx.x * kGradCols >= C) return;
    const int slot = blockIdx.y;
    const int rank = slot < snap.max_slots ? (int)snap.rank[slot] : 0;
    if (rank == 0) return;
    const int mtiles = (rank + 15) >> 4;   // 16-row groups of j
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = blockIdx.x * kGradCols;
    const int ncols = min(kGradCols, C - c0);
    float acc[4][2][4];   // [16-row group of j][8-column tile][fragment]
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int n = 0; n < 2; ++n) acc[a][n][0] = acc[a][n][1] = acc[a][n][2] = acc[a][n][3] = 0.f;
    const uint32_t smem = (uint32_t)__cvta_generic_to_shared(grad_smem);
    auto q_off = [](int buf) { return (uint32_t)(buf * (kGradQBytes + kGradPBytes)); };
    auto p_off = [](int buf) { return (uint32_t)(buf * (kGradQBytes + kGradPBytes) + kGradQBytes); };

    // Work items of this CTA: the slot's segments in order, each tile of a segment in order.  A piece block
    // (tile m, segment g) holds the rows of tile m that belong to g and zeros elsewhere, so the whole tile
    // of Q is multiplied (rows past T are zero-filled here).  Block and tile are brought into shared memory
    // by asynchronous copies, one item ahead of the arithmetic.
    int g = -1, m = 0, m_last = -1;
    auto advance = [&]() -> bool {   // next (g, m); false when the slot has no more
        if (m < m_last) { ++m; return true; }
        for (++g; g < G; ++g) {
            if (__ldg(slot_ids + g) != slot) continue;
            const int s0 = max(__ldg(seg_offsets + g), 0), s1 = min(__ldg(seg_offsets + g + 1), T);
            if (s1 <= s0) continue;
            m = s0 / kTileM;
            m_last = (s1 - 1) / kTileM;
            return true;
        }
        return false;
    };
    auto issue = [&](int buf) {
        const char* blk = reinterpret_cast<const char*>(pieces + (size_t)(m + g) * kTileM * kRankPad);
        for (int i = tid; i < kTileM * (kRankPad / 8); i += 256) {
            const int r = i / (kRankPad / 8), ch = i % (kRankPad / 8);
            grad_cp_async_16(smem + p_off(buf) + r * kGradPPitch + ch * 16, blk + (size_t)i * 16);
        }
        const int rows = min(kTileM, T - m * kTileM);
        const int chunks = ncols / 8;   // 16-byte chunks per row
        for (int i = tid; i < kTileM * chunks; i += 256) {
            const int r = i / chunks, ch = i % chunks;
            const uint32_t dst = smem + q_off(buf) + r * kGradQPitch + ch * 16;
            if (r < rows) grad_cp_async_16(dst, Q + (size_t)(m * kTileM + r) * C + c0 + ch * 8);
            else asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(dst), "r"(0u) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    bool have = advance();
    int buf = 0;
    if (have) issue(0);
    while (have) {
        const bool more = advance();
        if (more) issue(buf ^ 1);
        if (more) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();   // everybody's copies of the current item have landed
        const uint32_t qb = smem + q_off(buf), pb = smem + p_off(buf);
        // ldmatrix x4: lanes 0-7 address the rows of matrix 0, 8-15 of matrix 1, 16-23 of matrix 2, 24-31 of 3
        const int mi = lane >> 3, rr = lane & 7;
#pragma unroll 2
        for (int ks = 0; ks < kTileM / 16; ++ks) {
            const int p0 = ks * 16;
            // B operand for the warp's two column tiles: matrices (p 0-7 | 8-15) x (tile 0 | tile 1)
            uint32_t bq[2][2];
            {
                const uint32_t addr = qb + (uint32_t)((p0 + (mi & 1) * 8 + rr) * kGradQPitch + (warp * 16 + (mi >> 1) * 8) * 2);
                ldmatrix_x4_trans(addr, bq[0][0], bq[0][1], bq[1][0], bq[1][1]);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                if (a < mtiles) {
                    // A operand (j x p) from the block stored [p][j]: matrices (p 0-7, j 0-7), (p 0-7, j 8-15),
                    // (p 8-15, j 0-7), (p 8-15, j 8-15) give a0..a3
                    uint32_t a0, a1, a2, a3;
                    const uint32_t addr = pb + (uint32_t)((p0 + (mi >> 1) * 8 + rr) * kGradPPitch + (a * 16 + (mi & 1) * 8) * 2);
                    ldmatrix_x4_trans(addr, a0, a1, a2, a3);
#pragma unroll
                    for (int n = 0; n < 2; ++n) mma_bf16_16816(acc[a][n], a0, a1, a2, a3, bq[n][0], bq[n][1]);
                }
            }
        }
        __syncthreads();   // the buffer may be refilled two items from now
        have = more;
        buf ^= 1;
    }
    // fragment: c0,c1 = (j = gq, columns 2tq, 2tq+1), c2,c3 = (j = gq + 8, same columns)
    const int gq = lane >> 2, tq = lane & 3;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        if (a >= mtiles) continue;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = a * 16 + gq + (e >> 1) * 8;
                const int c = c0 + warp * 16 + n * 8 + tq * 2 + (e & 1);
                if (j < rank && c < C) {
                    float* o = mode == 0 ? out + ((size_t)slot * kRankPad + j) * C + c : out + ((size_t)slot * C + c) * kRankPad + j;
                    *o += acc[a][n][e];
                }
            }
        }
    }
}

cudaError_t launch_weight_grad(const SlotSnapshot& snap, const __nv_bfloat16* pieces, const void* Q, int T, int C,
                               const int32_t* seg_offsets, const int32_t* slot_ids, int G, float* out, int mode,
                               cudaStream_t stream, const __nv_bfloat16* pieces2, const void* Q2, int C2, float* out2, int mode2)
{
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    const int cmax = (out2 && C2 > C) ? C2 : C;
    pdl_config(cfg, attr, dim3((cmax + kGradCols - 1) / kGradCols, snap.max_slots, out2 ? 2 : 1), dim3(256), kGradSmemBytes, stream);
    const GradJob j0 = {pieces, (const __nv_bfloat16*)Q, out, C, mode};
    const GradJob j1 = {pieces2, (const __nv_bfloat16*)Q2, out2, C2, mode2};
    return cudaLaunchKernelEx(&cfg, weight_grad_kernel, snap, j0, j1, T, seg_offsets, slot_ids, G);
}

cudaError_t aux_init()   // called with the table's device current, once per table
{
    return cudaFuncSetAttribute(weight_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGradSmemBytes);
}

}  // namespace lml
