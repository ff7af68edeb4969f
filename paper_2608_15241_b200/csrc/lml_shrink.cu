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
// two MMAs.  Each CTA owns 16 rows of one piece; its 4 warps split K and are summed in a
// fixed order in shared memory (deterministic).
#include "lml_internal.cuh"

namespace lml {

constexpr int kShrinkWarps = 4;
constexpr int kShrinkRows = 16;

__global__ void __launch_bounds__(kShrinkWarps * 32) shrink_pieces_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaA,
    uint32_t* __restrict__ status, const __nv_bfloat16* __restrict__ x, int T, int K,
    const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ slot_ids, int G,
    const int32_t* __restrict__ perm, PlanWord* __restrict__ plan, __nv_bfloat16* __restrict__ u_blocks,
    int num_tiles)
{
    __shared__ float red[kShrinkWarps][kShrinkRows][kRankPad + 2];
    __shared__ int sh_piece[4];   // slot, lo, hi, found

    const int b = blockIdx.y, sub = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // One CTA validates the segment arrays for the whole call.
    if (b == 0 && sub == 0) {
        int bad_off = 0, bad_slot = 0;
        for (int g = tid; g < G; g += blockDim.x) {
            int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1);
            if (s1 < s0 || s0 < 0 || s1 > T) bad_off = 1;
            int s = __ldg(slot_ids + g);
            if (s != -1 && slot_rank(snap, s) == 0) bad_slot = 1;
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
    if (tid == 0) {
        int lo = 0, hi = G;   // invariant: candidates in [lo, hi)
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (mid + (__ldg(seg_offsets + mid) / kTileM) <= b) lo = mid; else hi = mid;
        }
        int g = lo, found = 0, slot = -1, plo = 0, phi = 0;
        if (G > 0) {
            int m = b - g;
            int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1);
            if (m >= 0 && m < num_tiles) {
                plo = max(max(s0, m * kTileM), 0);
                phi = min(min(s1, (m + 1) * kTileM), T);
                slot = __ldg(slot_ids + g);
                found = (plo < phi) && slot_rank(snap, slot) > 0;
            }
        }
        sh_piece[0] = slot; sh_piece[1] = plo; sh_piece[2] = phi; sh_piece[3] = found;
    }
    __syncthreads();
    if (!sh_piece[3]) return;
    const int slot = sh_piece[0], plo = sh_piece[1], phi = sh_piece[2];
    const int m = plo / kTileM;
    const int rank = snap.rank[slot];
    const int nblk = (rank + 7) >> 3;
    const int p0 = m * kTileM + sub * kShrinkRows;
    uint4* out = reinterpret_cast<uint4*>(u_blocks + ((size_t)b * kTileM + sub * kShrinkRows) * kRankPad);

    if (p0 + kShrinkRows <= plo || p0 >= phi) {   // no row of this sub-block is in the piece
        out[tid] = make_uint4(0, 0, 0, 0);        // 16 rows x 128 B = 128 x 16 B
        return;
    }

    const int gq = lane >> 2, tq = lane & 3;
    int pa = p0 + gq, pb = p0 + gq + 8;
    bool va = pa >= plo && pa < phi, vb = pb >= plo && pb < phi;
    if (perm) {
        bool badp = false;
        if (va) { pa = __ldg(perm + pa); if (pa < 0 || pa >= T) { va = false; badp = true; } }
        if (vb) { pb = __ldg(perm + pb); if (pb < 0 || pb >= T) { vb = false; badp = true; } }
        if (badp) atomicOr(status, LML_FLAG_BAD_PERM);
    }
    const __nv_bfloat16* xa = x + (size_t)(va ? pa : 0) * K;
    const __nv_bfloat16* xb = x + (size_t)(vb ? pb : 0) * K;
    const __nv_bfloat16* Abase = arenaA + ((size_t)slot * kRankPad + gq) * K;

    float acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

    const int steps = (K + 31) >> 5;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll 2
    for (int s = warp; s < steps; s += kShrinkWarps) {
        const int k = s * 32 + tq * 8;
        const bool kv = k < K;
        uint4 ra = (va && kv) ? ldg_nc_v4(xa + k) : zero4;
        uint4 rb = (vb && kv) ? ldg_nc_v4(xb + k) : zero4;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            if (nb < nblk) {
                uint4 w = kv ? ldg_nc_v4(Abase + (size_t)nb * 8 * K + k) : zero4;
                mma_bf16_16816(acc[nb], ra.x, rb.x, ra.y, rb.y, w.x, w.y);
                mma_bf16_16816(acc[nb], ra.z, rb.z, ra.w, rb.w, w.z, w.w);
            }
        }
    }

#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
        if (nb < nblk) {
            red[warp][gq][nb * 8 + tq * 2] = acc[nb][0];
            red[warp][gq][nb * 8 + tq * 2 + 1] = acc[nb][1];
            red[warp][gq + 8][nb * 8 + tq * 2] = acc[nb][2];
            red[warp][gq + 8][nb * 8 + tq * 2 + 1] = acc[nb][3];
        }
    }
    __syncthreads();
    {
        const int row = tid >> 3, c0 = (tid & 7) * 8;
        const float sc = snap.scale[slot];
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float s = 0.f;
            if (c0 + i < nblk * 8) {
#pragma unroll
                for (int w = 0; w < kShrinkWarps; ++w) s += red[w][row][c0 + i];
            }
            v[i] = s * sc;
        }
        uint4 o;
        o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]);
        o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
        out[row * 8 + (tid & 7)] = o;
    }
}

cudaError_t launch_shrink_pieces(const Arena& ar, const SlotSnapshot& snap, const void* x, int T,
                                 int d_in, const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                                 const int32_t* perm, PlanWord* plan, __nv_bfloat16* u_blocks,
                                 cudaStream_t stream)
{
    const int num_tiles = (T + kTileM - 1) / kTileM;
    dim3 grid(kTileM / kShrinkRows, num_tiles + G);
    shrink_pieces_kernel<<<grid, kShrinkWarps * 32, 0, stream>>>(
        snap, ar.A, ar.status, (const __nv_bfloat16*)x, T, d_in, seg_offsets, slot_ids, G, perm, plan,
        u_blocks, num_tiles);
    return cudaGetLastError();
}

}  // namespace lml
