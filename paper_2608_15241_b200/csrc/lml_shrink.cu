// LoRA shrink for the prefill path: u = scale_s * (x . A_s^T), written as bf16 "piece blocks"
// that the GEMM kernel consumes as extra tensor-core K-steps.
//
// A piece is the intersection of a 128-row tile m with a segment g whose slot is live.  Its
// block index is b = m + g, which is unique because segments are ordered row ranges: a later
// segment cannot reach into an earlier tile.  Block b holds 128 x 64 bf16: row i is
// scale * x[m*128+i] . A_s^T (columns >= rank are zero) when that row belongs to segment g
// and zero otherwise, so one UMMA of the whole block with B_s adds exactly the segment's LoRA
// term to the tile.
//
// The contraction runs on mma.sync m16n8k16 with operands loaded straight from global memory
// by 128-bit loads: a dot product does not care about the order of k, so lane (g, t) takes
// the 8 consecutive k at offset 8t of each 32-wide step for both operands and feeds them to
// two MMAs.  The pass is bound by reading x once, so what matters is bytes in flight: a
// thread-block cluster of up to 8 CTAs splits K for one 32-row slab of a piece, every warp
// issues all the loads of four steps before its first MMA, and the partial sums are combined
// in a fixed order — warps through shared memory, CTAs through distributed shared memory — so
// the result is deterministic and needs no scratch in global memory.
#include <cstdlib>
#include <cooperative_groups.h>

#include "lml_internal.cuh"
#include "lml_ptx_sm100.cuh"

namespace cg = cooperative_groups;

namespace lml {

constexpr int kShrinkWarps = 8;
constexpr int kShrinkRows = 32;       // rows of one CTA (two 16-row MMA tiles)
constexpr int kShrinkUnroll = 4;
constexpr int kShrinkMaxCluster = 8;
constexpr int kShrinkSegCache = 256;

template <int NB> struct ShrinkSmem {
    static constexpr int kCols = NB * 8;
    static constexpr int kPitch = kCols + 2;
    static constexpr int kBytes = (kShrinkWarps * kShrinkRows * kPitch + kShrinkRows * kCols) * 4;
};

// NB = number of 8-column blocks of u that can be non-zero (rank <= 8 * NB).
template <int NB>
__global__ void __launch_bounds__(kShrinkWarps * 32, NB <= 2 ? 2 : 1) shrink_pieces_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaA,
    uint32_t* __restrict__ status, const __nv_bfloat16* __restrict__ x, int T, int K,
    const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ slot_ids, int G,
    const __nv_bfloat16* __restrict__ x_in_place, const int32_t* __restrict__ tile_identity,
    PlanWord* __restrict__ plan, __nv_bfloat16* __restrict__ u_blocks, int num_tiles, int chained,
    __nv_bfloat16* __restrict__ u_blocks_neg)   // optional second copy of the blocks with the sign flipped
{
    // chained 0: launched with a full dependency on the work before it, so nothing to wait for; the GEMM that
    // follows may start its main loop right away.  chained 1: this is a further shrink pass of the same call,
    // launched as a programmatic dependent of the first, which had that full dependency: the passes run side by
    // side; one CTA then stays until the pass before is complete, so that whoever waits for this grid has
    // waited for all of them.  chained 2: the predecessor is the call's own short row-gather kernel; launched
    // as its programmatic dependent (the launch latency hides behind it), every CTA waits for it here before
    // it lets the GEMM go, so that the GEMM finds the gathered rows complete as well.
    if (chained == 2) ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    extern __shared__ float shrink_smem[];
    using S = ShrinkSmem<NB>;
    float* red = shrink_smem;                                           // [warp][row][pitch]
    float* partial = shrink_smem + kShrinkWarps * kShrinkRows * S::kPitch;   // [row][cols]
    __shared__ int sh_piece[4];   // slot, lo, hi, found
    __shared__ int seg_s[kShrinkSegCache + 1];   // the segment offsets, when they fit: the search below is then one round trip to memory, not one per step

    cg::cluster_group cluster = cg::this_cluster();
    const int KS = (int)gridDim.z, ks = (int)blockIdx.z;
    const int b = blockIdx.y, sub = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // One CTA validates the segment arrays for the whole call.
    if (b == 0 && sub == 0 && ks == 0) {
        if (chained == 1 && tid == 0) ptx::grid_dependency_wait();
        int bad_off = 0, bad_slot = 0;
        for (int g = tid; g < G; g += blockDim.x) {
            int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1);
            if (s1 < s0 || s0 < 0 || s1 > T) bad_off = 1;
            int s = __ldg(slot_ids + g);
            if (s != -1 && s1 > s0 && slot_rank(snap, s) == 0) bad_slot = 1;   // an empty segment may name anything
        }
        if (tid == 0 && (__ldg(seg_offsets) != 0 || __ldg(seg_offsets + G) != T)) bad_off = 1;
        bad_off = __syncthreads_or(bad_off);
        bad_slot = __syncthreads_or(bad_slot);
        if (tid == 0) {
            plan->lora_ok = bad_off ? 0 : 1;
            unsigned f = (bad_off ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_slot ? LML_FLAG_BAD_SLOT : 0u);
            if (f) atomicOr(status, f);
        }
    }

    // Which piece, if any, has block index b?  Largest g with g + tile_first(g) <= b.
    const bool seg_cached = G <= kShrinkSegCache;
    if (seg_cached) {
        for (int g = tid; g <= G; g += blockDim.x) seg_s[g] = __ldg(seg_offsets + g);
        __syncthreads();
    }
    if (tid == 0) {
        int lo = 0, hi = G;   // invariant: candidates in [lo, hi)
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            const int off = seg_cached ? seg_s[mid] : __ldg(seg_offsets + mid);
            if (mid + (off / kTileM) <= b) lo = mid; else hi = mid;
        }
        int g = lo, found = 0, slot = -1, plo = 0, phi = 0;
        if (G > 0) {
            int m = b - g;
            int s0 = seg_cached ? seg_s[g] : __ldg(seg_offsets + g), s1 = seg_cached ? seg_s[g + 1] : __ldg(seg_offsets + g + 1);
            if (m >= 0 && m < num_tiles) {
                plo = max(max(s0, m * kTileM), 0);
                phi = min(min(s1, (m + 1) * kTileM), T);
                slot = __ldg(slot_ids + g);
                const int r = slot_rank(snap, slot);
                found = (plo < phi) && r > 0 && r <= NB * 8;
            }
        }
        sh_piece[0] = slot; sh_piece[1] = plo; sh_piece[2] = phi; sh_piece[3] = found;
    }
    __syncthreads();
    // Every CTA of a cluster shares (b, sub) and therefore takes the same exits below.
    if (!sh_piece[3]) return;
    const int slot = sh_piece[0], plo = sh_piece[1], phi = sh_piece[2];
    const int m = plo / kTileM;
    const int nblk = ((int)snap.rank[slot] + 7) >> 3;
    const int p0 = m * kTileM + sub * kShrinkRows;
    uint4* out = reinterpret_cast<uint4*>(u_blocks + ((size_t)b * kTileM + sub * kShrinkRows) * kRankPad);
    uint4* out_neg = u_blocks_neg ? reinterpret_cast<uint4*>(u_blocks_neg + ((size_t)b * kTileM + sub * kShrinkRows) * kRankPad) : nullptr;

    if (p0 + kShrinkRows <= plo || p0 >= phi) {   // no row of this slab is in the piece
        if (ks == 0) {   // 32 rows x 128 B = 256 x 16 B
            out[tid] = make_uint4(0, 0, 0, 0);
            if (out_neg) out_neg[tid] = make_uint4(0, 0, 0, 0);
        }
        return;
    }

    const int gq = lane >> 2, tq = lane & 3;
    const __nv_bfloat16* xsrc = (tile_identity && __ldg(tile_identity + m)) ? x_in_place : x;   // in-place tiles were never copied
    const __nv_bfloat16* xr[4];
    bool xv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = p0 + gq + 8 * i;
        xv[i] = p >= plo && p < phi;
        xr[i] = xsrc + (size_t)(xv[i] ? p : 0) * K + tq * 8;
    }
    const __nv_bfloat16* Abase = arenaA + ((size_t)slot * kRankPad + gq) * K + tq * 8;

    float acc[2][NB][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) acc[h][nb][0] = acc[h][nb][1] = acc[h][nb][2] = acc[h][nb][3] = 0.f;

    const int steps = (K + 31) >> 5;
    const int stride = KS * kShrinkWarps;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    for (int s0 = ks * kShrinkWarps + warp; s0 < steps; s0 += stride * kShrinkUnroll) {
        uint4 xa[kShrinkUnroll][4];
#pragma unroll
        for (int i = 0; i < kShrinkUnroll; ++i) {
            const int k = (s0 + i * stride) * 32;
            const bool kv = k + tq * 8 < K;   // also false for steps past the end
#pragma unroll
            for (int r = 0; r < 4; ++r) xa[i][r] = (xv[r] && kv) ? ldg_nc_v4(xr[r] + k) : zero4;
        }
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            if (nb < nblk) {
                uint4 w[kShrinkUnroll];
#pragma unroll
                for (int i = 0; i < kShrinkUnroll; ++i) {
                    const int k = (s0 + i * stride) * 32;
                    w[i] = (k + tq * 8 < K) ? ldg_nc_v4(Abase + (size_t)nb * 8 * K + k) : zero4;
                }
#pragma unroll
                for (int i = 0; i < kShrinkUnroll; ++i) {
                    mma_bf16_16816(acc[0][nb], xa[i][0].x, xa[i][1].x, xa[i][0].y, xa[i][1].y, w[i].x, w[i].y);
                    mma_bf16_16816(acc[0][nb], xa[i][0].z, xa[i][1].z, xa[i][0].w, xa[i][1].w, w[i].z, w[i].w);
                    mma_bf16_16816(acc[1][nb], xa[i][2].x, xa[i][3].x, xa[i][2].y, xa[i][3].y, w[i].x, w[i].y);
                    mma_bf16_16816(acc[1][nb], xa[i][2].z, xa[i][3].z, xa[i][2].w, xa[i][3].w, w[i].z, w[i].w);
                }
            }
        }
    }

    // warps -> CTA partial, fixed order
    float* myred = red + warp * kShrinkRows * S::kPitch;
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            const int c = nb * 8 + tq * 2;
            myred[(h * 16 + gq) * S::kPitch + c] = acc[h][nb][0];
            myred[(h * 16 + gq) * S::kPitch + c + 1] = acc[h][nb][1];
            myred[(h * 16 + gq + 8) * S::kPitch + c] = acc[h][nb][2];
            myred[(h * 16 + gq + 8) * S::kPitch + c + 1] = acc[h][nb][3];
        }
    __syncthreads();
    for (int e = tid; e < kShrinkRows * S::kCols; e += kShrinkWarps * 32) {
        const int row = e / S::kCols, col = e % S::kCols;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kShrinkWarps; ++w) s += red[(w * kShrinkRows + row) * S::kPitch + col];
        partial[e] = s;
    }
    cluster.sync();
    if (ks == 0) {   // CTAs -> result, fixed order, through distributed shared memory
        const int row = tid >> 3, c0 = (tid & 7) * 8;
        const float sc = snap.scale[slot];
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
        if (c0 < S::kCols) {
            for (int r = 0; r < KS; ++r) {
                const float* peer = cluster.map_shared_rank(partial, r) + row * S::kCols + c0;
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] += peer[i];
            }
        }
        uint4 o;
        o.x = pack_bf16(v[0] * sc, v[1] * sc); o.y = pack_bf16(v[2] * sc, v[3] * sc);
        o.z = pack_bf16(v[4] * sc, v[5] * sc); o.w = pack_bf16(v[6] * sc, v[7] * sc);
        out[row * 8 + (tid & 7)] = o;
        if (out_neg) out_neg[row * 8 + (tid & 7)] = make_uint4(o.x ^ 0x80008000u, o.y ^ 0x80008000u, o.z ^ 0x80008000u, o.w ^ 0x80008000u);
    }
    cluster.sync();   // peers stay alive until their partials have been read
}

template <int NB>
static cudaError_t launch_shrink_nb(const Arena& ar, const SlotSnapshot& snap, const void* x, int T, int d_in,
                                    const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                                    const void* x_in_place, const int32_t* tile_identity, PlanWord* plan,
                                    __nv_bfloat16* u_blocks, cudaStream_t stream, int chained, __nv_bfloat16* u_blocks_neg)
{
    const int num_tiles = (T + kTileM - 1) / kTileM;
    int ks = (d_in + 1023) / 1024;
    ks = ks < 1 ? 1 : (ks > kShrinkMaxCluster ? kShrinkMaxCluster : ks);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kTileM / kShrinkRows, num_tiles + G, ks);
    cfg.blockDim = dim3(kShrinkWarps * 32);
    cfg.dynamicSmemBytes = ShrinkSmem<NB>::kBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = ks;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 2 : 1;
    const __nv_bfloat16* arenaA = ar.A;
    uint32_t* status = ar.status;
    const __nv_bfloat16* xb = (const __nv_bfloat16*)x;
    const __nv_bfloat16* xip = (const __nv_bfloat16*)x_in_place;
    return cudaLaunchKernelEx(&cfg, shrink_pieces_kernel<NB>, snap, arenaA, status, xb, T, d_in, seg_offsets,
                              slot_ids, G, xip, tile_identity, plan, u_blocks, num_tiles, chained, u_blocks_neg);
}

cudaError_t shrink_init()
{
    cudaError_t e = cudaFuncSetAttribute(shrink_pieces_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ShrinkSmem<2>::kBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(shrink_pieces_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                ShrinkSmem<8>::kBytes);
}

cudaError_t launch_shrink_pieces(const Arena& ar, const SlotSnapshot& snap, const void* x, int T,
                                 int d_in, const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                                 const void* x_in_place, const int32_t* tile_identity, PlanWord* plan,
                                 __nv_bfloat16* u_blocks, cudaStream_t stream, int chained, __nv_bfloat16* u_blocks_neg)
{
    int max_rank = 0;
    for (int i = 0; i < snap.max_slots; ++i) max_rank = snap.rank[i] > max_rank ? snap.rank[i] : max_rank;
    if (max_rank <= 16)
        return launch_shrink_nb<2>(ar, snap, x, T, d_in, seg_offsets, slot_ids, G, x_in_place, tile_identity, plan, u_blocks, stream, chained, u_blocks_neg);
    return launch_shrink_nb<8>(ar, snap, x, T, d_in, seg_offsets, slot_ids, G, x_in_place, tile_identity, plan, u_blocks, stream, chained, u_blocks_neg);
}

}  // namespace lml
