// Decode path (T <= 16 tokens): bandwidth-bound.  W0 is read exactly once with 128-bit loads.
//
// Two kernels, chained with programmatic dependent launch so the second one starts streaming W0
// while the first (tiny) one is still running:
//   decode_shrink_kernel  u[row][j] = scale_s * sum_k x[row][k] A_s[j][k]  (fp32, one warp per
//                         (token, j)), plus the slot of every row.
//   decode_main_kernel    each CTA owns 16 rows of W0 (16 output columns).  y^T = W0 . x^T runs on
//                         mma.sync m16n8k16 with W0 as the 16-row operand and the tokens as the
//                         8-wide operand; both come straight from global memory in 16-byte
//                         pieces (the k order inside a 32-wide step is permuted identically for
//                         both operands, which a dot product does not see).  The CTA's 8 warps
//                         split K and are summed in a fixed order; the LoRA expand
//                         sum_j u[t][j] B_s[n][j] is added in fp32 before the single bf16 rounding.
#include "lml_internal.cuh"
#include "lml_ptx_sm100.cuh"

namespace lml {

constexpr int kDecWarps = 8;
constexpr int kDecRows = 16;     // W0 rows per CTA
constexpr int kDecUnroll = 4;

__global__ void __launch_bounds__(256) decode_shrink_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaA,
    uint32_t* __restrict__ status, const __nv_bfloat16* __restrict__ x, int T, int K,
    const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ slot_ids, int G,
    const int32_t* __restrict__ perm, float* __restrict__ u, int32_t* __restrict__ row_slot)
{
    ptx::grid_launch_dependents();   // the main kernel may start streaming W0 right away
    __shared__ int sh[2];            // row, slot
    const int pos = blockIdx.x, jb = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // every CTA checks the segment arrays itself (G is small next to the work that follows)
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
        unsigned f = (bad_off ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_slot ? LML_FLAG_BAD_SLOT : 0u);
        int row = pos, slot = -1;
        if (perm) {
            row = __ldg(perm + pos);
            if (row < 0 || row >= T) { row = -1; f |= LML_FLAG_BAD_PERM; }
        }
        if (!bad_off && row >= 0) {
            int g = seg_upper(seg_offsets, G, pos);
            if (g < G) {
                int s = __ldg(slot_ids + g);
                if (slot_rank(snap, s) > 0) slot = s;
            }
        }
        if (f && pos == 0 && jb == 0) atomicOr(status, f);
        sh[0] = row; sh[1] = slot;
        if (jb == 0 && row >= 0) row_slot[row] = slot;
    }
    __syncthreads();
    const int row = sh[0], slot = sh[1];
    if (row < 0) return;
    const int j = jb * kDecWarps + warp;
    float dot = 0.f;
    if (slot >= 0 && j < (int)snap.rank[slot]) {
        const __nv_bfloat16* xr = x + (size_t)row * K;
        const __nv_bfloat16* ar = arenaA + ((size_t)slot * kRankPad + j) * K;
        for (int k = lane * 8; k < K; k += 256) {
            uint4 a = ldg_nc_v4(xr + k), b = ldg_nc_v4(ar + k);
            dot = fmaf(bf16_lo(a.x), bf16_lo(b.x), dot); dot = fmaf(bf16_hi(a.x), bf16_hi(b.x), dot);
            dot = fmaf(bf16_lo(a.y), bf16_lo(b.y), dot); dot = fmaf(bf16_hi(a.y), bf16_hi(b.y), dot);
            dot = fmaf(bf16_lo(a.z), bf16_lo(b.z), dot); dot = fmaf(bf16_hi(a.z), bf16_hi(b.z), dot);
            dot = fmaf(bf16_lo(a.w), bf16_lo(b.w), dot); dot = fmaf(bf16_hi(a.w), bf16_hi(b.w), dot);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        dot *= snap.scale[slot];
    }
    if (lane == 0) u[row * kRankPad + j] = dot;
}

template <bool kTwoBlocks>   // false: T <= 8 (one 8-token MMA block), true: T <= 16
__global__ void __launch_bounds__(kDecWarps * 32) decode_main_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaB,
    const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ W0,
    __nv_bfloat16* __restrict__ y, const float* __restrict__ u, const int32_t* __restrict__ row_slot,
    int T, int K, int N, int has_lora)
{
    __shared__ float red[kDecWarps][kDecRows][17];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const int n0 = blockIdx.x * kDecRows;
    const int na = n0 + gq, nb = n0 + gq + 8;
    const bool va = na < N, vb = nb < N;
    const __nv_bfloat16* wa = W0 + (size_t)(va ? na : 0) * K + tq * 8;
    const __nv_bfloat16* wb = W0 + (size_t)(vb ? nb : 0) * K + tq * 8;
    const bool ta = gq < T, tb = kTwoBlocks && (gq + 8 < T);
    const __nv_bfloat16* xa = x + (size_t)(ta ? gq : 0) * K + tq * 8;
    const __nv_bfloat16* xb = x + (size_t)(tb ? gq + 8 : 0) * K + tq * 8;

    float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    const int steps = (K + 31) >> 5;
    for (int s0 = warp; s0 < steps; s0 += kDecWarps * kDecUnroll) {
        uint4 ra[kDecUnroll], rb[kDecUnroll], qa[kDecUnroll], qb[kDecUnroll];
#pragma unroll
        for (int i = 0; i < kDecUnroll; ++i) {
            const int k = (s0 + i * kDecWarps) * 32;
            const bool kv = (k + tq * 8) < K;   // also false for steps past the end
            ra[i] = (va && kv) ? ldg_nc_v4(wa + k) : zero4;
            rb[i] = (vb && kv) ? ldg_nc_v4(wb + k) : zero4;
            qa[i] = (ta && kv) ? __ldg(reinterpret_cast<const uint4*>(xa + k)) : zero4;
            if (kTwoBlocks) qb[i] = (tb && kv) ? __ldg(reinterpret_cast<const uint4*>(xb + k)) : zero4;
        }
#pragma unroll
        for (int i = 0; i < kDecUnroll; ++i) {
            mma_bf16_16816(acc0, ra[i].x, rb[i].x, ra[i].y, rb[i].y, qa[i].x, qa[i].y);
            mma_bf16_16816(acc0, ra[i].z, rb[i].z, ra[i].w, rb[i].w, qa[i].z, qa[i].w);
            if (kTwoBlocks) {
                mma_bf16_16816(acc1, ra[i].x, rb[i].x, ra[i].y, rb[i].y, qb[i].x, qb[i].y);
                mma_bf16_16816(acc1, ra[i].z, rb[i].z, ra[i].w, rb[i].w, qb[i].z, qb[i].w);
            }
        }
    }
    // fragment -> red[warp][W0 row][token]
    red[warp][gq][tq * 2] = acc0[0];     red[warp][gq][tq * 2 + 1] = acc0[1];
    red[warp][gq + 8][tq * 2] = acc0[2]; red[warp][gq + 8][tq * 2 + 1] = acc0[3];
    if (kTwoBlocks) {
        red[warp][gq][8 + tq * 2] = acc1[0];     red[warp][gq][8 + tq * 2 + 1] = acc1[1];
        red[warp][gq + 8][8 + tq * 2] = acc1[2]; red[warp][gq + 8][8 + tq * 2 + 1] = acc1[3];
    }
    __syncthreads();
    const int t = tid >> 4, i = tid & 15;
    if (t >= T || (!kTwoBlocks && t >= 8)) return;
    const int n = n0 + i;
    if (n >= N) return;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) v += red[w][i][t];
    if (has_lora) {
        ptx::grid_dependency_wait();   // u and row_slot come from the shrink kernel
        const int slot = row_slot[t];
        if (slot >= 0 && slot < snap.max_slots) {
            const int r8 = ((int)snap.rank[slot] + 7) >> 3;
            const uint4* bp = reinterpret_cast<const uint4*>(arenaB + ((size_t)slot * N + n) * kRankPad);
            const float4* up = reinterpret_cast<const float4*>(u + t * kRankPad);
            float d = 0.f;
            for (int c = 0; c < r8; ++c) {
                uint4 b = ldg_nc_v4(bp + c);
                float4 u0 = up[2 * c], u1 = up[2 * c + 1];
                d = fmaf(u0.x, bf16_lo(b.x), d); d = fmaf(u0.y, bf16_hi(b.x), d);
                d = fmaf(u0.z, bf16_lo(b.y), d); d = fmaf(u0.w, bf16_hi(b.y), d);
                d = fmaf(u1.x, bf16_lo(b.z), d); d = fmaf(u1.y, bf16_hi(b.z), d);
                d = fmaf(u1.z, bf16_lo(b.w), d); d = fmaf(u1.w, bf16_hi(b.w), d);
            }
            v += d;
        }
    }
    y[(size_t)t * N + n] = __float2bfloat16_rn(v);
}

cudaError_t launch_decode(const Arena& ar, const SlotSnapshot& snap, const DecodeArgs& a, cudaStream_t stream,
                          int* launches)
{
    const bool lora = a.G > 0;
    *launches = 0;
    if (lora) {
        dim3 grid(a.T, kRankPad / kDecWarps);
        decode_shrink_kernel<<<grid, 256, 0, stream>>>(snap, ar.A, ar.status, (const __nv_bfloat16*)a.x, a.T,
                                                       a.d_in, a.seg_offsets, a.slot_ids, a.G, a.perm, a.u,
                                                       a.row_slot);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((a.d_out + kDecRows - 1) / kDecRows);
    cfg.blockDim = dim3(kDecWarps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = lora ? 1 : 0;   // only overlap with our own shrink kernel, never with foreign work
    const __nv_bfloat16* xb = (const __nv_bfloat16*)a.x;
    const __nv_bfloat16* wb = (const __nv_bfloat16*)a.W0;
    __nv_bfloat16* yb = (__nv_bfloat16*)a.y;
    const float* up = a.u;
    const int32_t* rs = a.row_slot;
    const __nv_bfloat16* arenaB = ar.B;
    int has = lora ? 1 : 0;
    cudaError_t e;
    if (a.T <= 8)
        e = cudaLaunchKernelEx(&cfg, decode_main_kernel<false>, snap, arenaB, xb, wb, yb, up, rs, a.T, a.d_in, a.d_out, has);
    else
        e = cudaLaunchKernelEx(&cfg, decode_main_kernel<true>, snap, arenaB, xb, wb, yb, up, rs, a.T, a.d_in, a.d_out, has);
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace lml
