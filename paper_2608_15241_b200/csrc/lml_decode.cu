// Decode path (T <= 16 tokens): bandwidth-bound.  W0 is read exactly once.
//
// Two kernels, chained with programmatic dependent launch so the second one starts streaming W0
// while the first (tiny) one is still running:
//   decode_shrink_kernel  u[row][j] = scale_s * sum_k x[row][k] A_s[j][k]  (fp32, one warp per
//                         (token, j)).
//   decode_main_kernel    one persistent CTA per SM, each owning a contiguous, balanced range of
//                         W0 rows (N/148 of them, +-1), because an SM cannot take in much more than
//                         its fair share of HBM bandwidth and contiguous addresses stream best.
//                         A producer warp copies 8 rows x 1024 columns per stage (one 2 KB bulk
//                         asynchronous copy per row) into a shared-memory ring, unit after unit, so
//                         the CTA walks its rows front to back.
//                         Eight consumer warps each own a fixed slice of K: their x fragments are
//                         loaded once into registers and reused for every row.  y^T += W0.x^T runs on
//                         mma.sync m16n8k16 with the tokens as the 16-row operand (T <= 16 is exactly
//                         one tile) and 8 rows of W0 as the 8-wide operand.  The k order inside a
//                         32-wide step is permuted identically for both operands, which a dot product
//                         does not see, so operands are plain 16-byte loads.  Per-warp partial sums go
//                         to per-warp slots and are added in a fixed order; the LoRA expand
//                         sum_j u[t][j] B_s[n][j] is added in fp32 before the single bf16 rounding.
//                         d_in > 4096 is walked in spans of 4096 columns.  All waits are bounded.
#include "lml_internal.cuh"
#include "lml_ptx_sm100.cuh"

namespace lml {

using namespace ptx;

constexpr int kDecConsumers = 8;                 // consumer warps
constexpr int kDecThreads = (kDecConsumers + 1) * 32;
constexpr int kDecUnitRows = 8;                  // W0 rows per unit = the 8-wide MMA operand
constexpr int kDecSpan = 4096;                   // columns whose x fragments fit in registers (half of it for T > 8)
constexpr int kDecChunk = 2048;                  // columns per stage (one 4 KB bulk copy per row)
constexpr int kDecChunksPerSpan = kDecSpan / kDecChunk;             // 4
constexpr int kDecStepsPerChunk = kDecChunk / 32 / kDecConsumers;   // 4 k-steps per warp and stage
constexpr int kDecRowPitch = kDecChunk * 2 + 64; // bytes; a multiple of 16 that is 4 mod 8 in 16-byte chunks: rows land on different banks
constexpr int kDecStageBytes = kDecUnitRows * kDecRowPitch;
constexpr int kDecStages = 5;
constexpr int kDecRoundUnits = 6;                // units (= 48 rows) reduced together
constexpr int kDecSlotFloats = 16 * kDecUnitRows;   // [token][row] partial sums of one warp for one unit
constexpr int kDecSlotBytes = kDecRoundUnits * kDecConsumers * kDecSlotFloats * 4;
constexpr int kDecUBytes = 16 * kRankPad * 4;     // shared-memory copy of u for the epilogue
constexpr int kDecSmemBytes = 128 + kDecStages * kDecStageBytes + kDecSlotBytes + kDecUBytes + 256;
static_assert(kDecSmemBytes <= 232448, "shared memory budget");

struct DecCtrl {
    uint64_t full[kDecStages];
    uint64_t empty[kDecStages];
    int abort;
    int bad_offsets;
    int slot_of_row[16];
};
static_assert(sizeof(DecCtrl) <= 256, "control block");

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void prefetch_l2(const void* p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

constexpr int kDecShrinkSegs = 256;   // segments looked up in one parallel pass

// Slot of position `pos` and validity of the segment arrays, found by the whole CTA in one round
// of loads (every thread looks at one segment) when G is small, else by binary search.
__device__ __forceinline__ void decode_lookup(const SlotSnapshot& snap, const int32_t* __restrict__ seg_offsets,
                                              const int32_t* __restrict__ slot_ids, int G, int T, int pos,
                                              int* sh_slot, int& bad_off, int& bad_slot)
{
    bad_off = 0; bad_slot = 0;
    const int tid = threadIdx.x;
    if (tid == 0) *sh_slot = -1;
    __syncthreads();
    for (int g = tid; g < G; g += blockDim.x) {
        const int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1), s = __ldg(slot_ids + g);
        if (s1 < s0 || s0 < 0 || s1 > T) bad_off = 1;
        if (g == 0 && s0 != 0) bad_off = 1;
        if (g == G - 1 && s1 != T) bad_off = 1;
        const int r = slot_rank(snap, s);
        if (s != -1 && r == 0) bad_slot = 1;
        if (pos >= s0 && pos < s1) *sh_slot = r > 0 ? s : -1;   // at most one segment holds pos when offsets are monotone
    }
    bad_off = __syncthreads_or(bad_off);
    bad_slot = __syncthreads_or(bad_slot);
}

// One CTA per (position, j): all 256 threads share one dot product, so a thread has only a couple
// of 16-byte loads of x and of A in flight and the whole kernel is two memory round trips long
// (segment lookup, then operands).  CTAs whose j is beyond the slot's rank only write a zero.
__global__ void __launch_bounds__(256) decode_shrink_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaA,
    uint32_t* __restrict__ status, const __nv_bfloat16* __restrict__ x, int T, int K,
    const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ slot_ids, int G,
    const int32_t* __restrict__ perm, float* __restrict__ u, int32_t* __restrict__ row_slot)
{
    grid_dependency_wait();     // work before this call is complete
    grid_launch_dependents();   // the main kernel may start streaming W0 right away
    __shared__ int sh_slot;
    __shared__ float sh_part[8];
    const int pos = blockIdx.x, j = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    int row = perm ? __ldg(perm + pos) : pos;   // in flight together with the segment lookup
    int bad_off, bad_slot;
    decode_lookup(snap, seg_offsets, slot_ids, G, T, pos, &sh_slot, bad_off, bad_slot);
    unsigned f = (bad_off ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_slot ? LML_FLAG_BAD_SLOT : 0u);
    if (row < 0 || row >= T) { row = -1; f |= LML_FLAG_BAD_PERM; }
    const int slot = (bad_off || row < 0) ? -1 : sh_slot;
    if (tid == 0 && j == 0) {
        if (f) atomicOr(status, f);
        if (row >= 0) row_slot[row] = slot;
    }
    if (row < 0) return;
    if (slot < 0 || j >= (int)snap.rank[slot]) {
        if (tid == 0) u[row * kRankPad + j] = 0.f;
        return;
    }
    const __nv_bfloat16* xr = x + (size_t)row * K;
    const __nv_bfloat16* ar = arenaA + ((size_t)slot * kRankPad + j) * K;
    float dot = 0.f;
    for (int k0 = tid * 8; k0 < K; k0 += 256 * 8 * 2) {
        const int k1 = k0 + 256 * 8;
        const bool v1 = k1 < K;
        const uint4 a0 = ldg_nc_v4(xr + k0), b0 = ldg_nc_v4(ar + k0);
        const uint4 a1 = v1 ? ldg_nc_v4(xr + k1) : make_uint4(0, 0, 0, 0);
        const uint4 b1 = v1 ? ldg_nc_v4(ar + k1) : make_uint4(0, 0, 0, 0);
        float d0 = 0.f, d1 = 0.f;
        d0 = fmaf(bf16_lo(a0.x), bf16_lo(b0.x), d0); d0 = fmaf(bf16_hi(a0.x), bf16_hi(b0.x), d0);
        d0 = fmaf(bf16_lo(a0.y), bf16_lo(b0.y), d0); d0 = fmaf(bf16_hi(a0.y), bf16_hi(b0.y), d0);
        d0 = fmaf(bf16_lo(a0.z), bf16_lo(b0.z), d0); d0 = fmaf(bf16_hi(a0.z), bf16_hi(b0.z), d0);
        d0 = fmaf(bf16_lo(a0.w), bf16_lo(b0.w), d0); d0 = fmaf(bf16_hi(a0.w), bf16_hi(b0.w), d0);
        d1 = fmaf(bf16_lo(a1.x), bf16_lo(b1.x), d1); d1 = fmaf(bf16_hi(a1.x), bf16_hi(b1.x), d1);
        d1 = fmaf(bf16_lo(a1.y), bf16_lo(b1.y), d1); d1 = fmaf(bf16_hi(a1.y), bf16_hi(b1.y), d1);
        d1 = fmaf(bf16_lo(a1.z), bf16_lo(b1.z), d1); d1 = fmaf(bf16_hi(a1.z), bf16_hi(b1.z), d1);
        d1 = fmaf(bf16_lo(a1.w), bf16_lo(b1.w), d1); d1 = fmaf(bf16_hi(a1.w), bf16_hi(b1.w), d1);
        dot += d0 + d1;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (lane == 0) sh_part[warp] = dot;
    __syncthreads();
    if (tid == 0) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += sh_part[w];
        u[row * kRankPad + j] = s * snap.scale[slot];
    }
}

template <bool kTwo>   // false: T <= 8, the second half of the 16-row MMA operand is zero and needs no registers
__global__ void __launch_bounds__(kDecThreads, 1) decode_main_kernel(
    const __grid_constant__ SlotSnapshot snap, const __nv_bfloat16* __restrict__ arenaB,
    const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ W0,
    __nv_bfloat16* __restrict__ y, const float* __restrict__ u, const int32_t* __restrict__ seg_offsets,
    const int32_t* __restrict__ slot_ids, const int32_t* __restrict__ perm, uint32_t* __restrict__ status,
    int T, int K, int N, int G)
{
    extern __shared__ uint8_t dec_smem_raw[];
    const uint32_t raw = smem_u32(dec_smem_raw);
    const uint32_t ring = (raw + 127u) & ~127u;
    uint8_t* base_ptr = dec_smem_raw + (ring - raw);
    float* slots = reinterpret_cast<float*>(base_ptr + kDecStages * kDecStageBytes);   // [stage][warp][token][row]
    float* u_s = reinterpret_cast<float*>(base_ptr + kDecStages * kDecStageBytes + kDecSlotBytes);   // [16][64]
    DecCtrl* ctrl = reinterpret_cast<DecCtrl*>(base_ptr + kDecStages * kDecStageBytes + kDecSlotBytes + kDecUBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // this CTA's rows: a contiguous, balanced range
    const int row_begin = (int)((long long)blockIdx.x * N / gridDim.x);
    const int row_end = (int)((long long)(blockIdx.x + 1) * N / gridDim.x);
    // x fragments of a span live in registers; with two 8-token blocks a span is half as wide, so
    // both variants hold 64 fragment registers and stay clear of spills
    constexpr int kSpan = kTwo ? kDecSpan / 2 : kDecSpan;
    constexpr int kChunksPerSpan = kSpan / kDecChunk;
    const int nspans = (K + kSpan - 1) / kSpan;

    if (tid == 0) {
        for (int s = 0; s < kDecStages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), kDecConsumers);
        }
        ctrl->abort = 0;
        ctrl->bad_offsets = 0;
        fence_mbar_init();
    }
    if (tid < 16) ctrl->slot_of_row[tid] = -1;
    if (G == 0) {   // no shrink kernel ran before this one: wait for foreign work here
        grid_dependency_wait();
        grid_launch_dependents();
    }
    __syncthreads();
    volatile int* abort = &ctrl->abort;

    const int gq = lane >> 2, tq = lane & 3;
    const bool consumer = warp < kDecConsumers;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    bool u_ready = false;

    // Consumer warp 0 works out the slot of every row of x (the same rule the shrink kernel
    // applies) and pulls the B rows this CTA will need into L2 while W0 streams.
    if (warp == 0 && G > 0) {
        int bad = 0;
        for (int g = lane; g < G; g += 32) {
            int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1);
            if (s1 < s0 || s0 < 0 || s1 > T) bad = 1;
        }
        if (lane == 0 && (__ldg(seg_offsets) != 0 || __ldg(seg_offsets + G) != T)) bad = 1;
        bad = __any_sync(0xffffffffu, bad);
        if (lane == 0) ctrl->bad_offsets = bad;
        if (!bad && lane < T) {
            int row = perm ? __ldg(perm + lane) : lane;
            if (row >= 0 && row < T) {
                int g = seg_upper(seg_offsets, G, lane);
                int slot = -1;
                if (g < G) { int s = __ldg(slot_ids + g); if (slot_rank(snap, s) > 0) slot = s; }
                ctrl->slot_of_row[row] = slot;
                if (slot >= 0) {
                    const char* b = reinterpret_cast<const char*>(arenaB + ((size_t)slot * N + row_begin) * kRankPad);
                    for (int r = 0; r < row_end - row_begin; ++r) prefetch_l2(b + (size_t)r * kRankPad * 2);
                }
            }
        }
    }

    for (int round_begin = row_begin; round_begin < row_end; round_begin += kDecRoundUnits * kDecUnitRows) {
        const int round_rows = min(kDecRoundUnits * kDecUnitRows, row_end - round_begin);
        const int nunits = (round_rows + kDecUnitRows - 1) / kDecUnitRows;
        for (int sp = 0; sp < nspans; ++sp) {
            const int k_begin = sp * kSpan;
            const int span = min(kSpan, K - k_begin);
            const int nchunks = (span + kDecChunk - 1) / kDecChunk;
            if (!consumer) {
                // ---------------------------------------------------------- producer warp
                // lane r < 8 copies this stage's 2 KB of row r; a unit's chunks follow each other, so the
                // CTA walks its rows front to back
                for (int un = 0; un < nunits && ok; ++un) {
                    const int r0 = round_begin + un * kDecUnitRows;
                    const int rows = min(kDecUnitRows, round_begin + round_rows - r0);
                    for (int kc = 0; kc < nchunks && ok; ++kc) {
                        const int cols = min(kDecChunk, span - kc * kDecChunk);
                        ok = mbar_wait_warp(smem_u32(&ctrl->empty[stage]), phase ^ 1u, abort);
                        if (!ok) break;
                        if (lane == 0) mbar_arrive_expect_tx(smem_u32(&ctrl->full[stage]), (uint32_t)(rows * cols * 2));
                        __syncwarp();
                        if (lane < rows)
                            bulk_copy_g2s(ring + stage * kDecStageBytes + lane * kDecRowPitch,
                                          W0 + (size_t)(r0 + lane) * K + k_begin + kc * kDecChunk,
                                          (uint32_t)(cols * 2), smem_u32(&ctrl->full[stage]));
                        if (++stage == kDecStages) { stage = 0; phase ^= 1u; }
                    }
                }
            } else {
                // ---------------------------------------------------------- consumer warps
                // this warp's k-steps of the span: chunk kc, steps warp*4 .. warp*4+3.  The x fragments
                // live in registers for every row of the round.
                uint4 xa[kChunksPerSpan * kDecStepsPerChunk], xc[kTwo ? kChunksPerSpan * kDecStepsPerChunk : 1];
                const bool ta = gq < T, tb = gq + 8 < T;
#pragma unroll
                for (int i = 0; i < kChunksPerSpan * kDecStepsPerChunk; ++i) {
                    const int c = (i / kDecStepsPerChunk) * kDecChunk + (warp * kDecStepsPerChunk + i % kDecStepsPerChunk) * 32 + tq * 8;
                    const bool lv = c < span;
                    xa[i] = (lv && ta) ? ldg_nc_v4(x + (size_t)gq * K + k_begin + c) : make_uint4(0, 0, 0, 0);
                    if (kTwo) xc[i] = (lv && tb) ? ldg_nc_v4(x + (size_t)(gq + 8) * K + k_begin + c) : make_uint4(0, 0, 0, 0);
                }
                for (int un = 0; un < nunits && ok; ++un) {
                    const int rows = min(kDecUnitRows, round_rows - un * kDecUnitRows);
                    const bool rv = gq < rows;   // lanes whose row of the 8-wide operand is real
                    // Four independent accumulator chains keep several MMAs in flight per warp.
                    float acc4[4][4];
#pragma unroll
                    for (int a = 0; a < 4; ++a) acc4[a][0] = acc4[a][1] = acc4[a][2] = acc4[a][3] = 0.f;
#pragma unroll
                    for (int kc = 0; kc < kChunksPerSpan; ++kc) {
                        if (kc < nchunks && ok) {
                            ok = mbar_wait_warp(smem_u32(&ctrl->full[stage]), phase, abort);
                            if (ok) {
                                const uint32_t wbase = ring + stage * kDecStageBytes + gq * kDecRowPitch + tq * 16;
#pragma unroll
                                for (int i = 0; i < kDecStepsPerChunk; ++i) {
                                    const int c0 = kc * kDecChunk + (warp * kDecStepsPerChunk + i) * 32;
                                    if (c0 < span) {   // uniform across the warp: all lanes issue the MMAs or none
                                        const uint4 w = (rv && c0 + tq * 8 < span)
                                                            ? lds128(wbase + (uint32_t)((warp * kDecStepsPerChunk + i) * 64))
                                                            : make_uint4(0, 0, 0, 0);
                                        const uint4 a0 = xa[kc * kDecStepsPerChunk + i];
                                        const uint4 a1 = kTwo ? xc[kc * kDecStepsPerChunk + i] : make_uint4(0, 0, 0, 0);
                                        mma_bf16_16816(acc4[(2 * i) & 3], a0.x, a1.x, a0.y, a1.y, w.x, w.y);
                                        mma_bf16_16816(acc4[(2 * i + 1) & 3], a0.z, a1.z, a0.w, a1.w, w.z, w.w);
                                    }
                                }
                                __syncwarp();
                                if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[stage]));
                                if (++stage == kDecStages) { stage = 0; phase ^= 1u; }
                            }
                        }
                    }
                    // fragment: c0,c1 = (token gq, rows 2tq, 2tq+1); c2,c3 = (token gq+8, same rows)
                    float* sl = slots + (un * kDecConsumers + warp) * kDecSlotFloats;
                    float vs[4];
#pragma unroll
                    for (int a = 0; a < 4; ++a)
                        vs[a] = (acc4[0][a] + acc4[1][a]) + (acc4[2][a] + acc4[3][a]);
                    const float v0 = vs[0], v1 = vs[1], v2 = vs[2], v3 = vs[3];
                    if (sp == 0) {
                        sl[gq * 8 + tq * 2] = v0;       sl[gq * 8 + tq * 2 + 1] = v1;
                        sl[(gq + 8) * 8 + tq * 2] = v2; sl[(gq + 8) * 8 + tq * 2 + 1] = v3;
                    } else {
                        sl[gq * 8 + tq * 2] += v0;       sl[gq * 8 + tq * 2 + 1] += v1;
                        sl[(gq + 8) * 8 + tq * 2] += v2; sl[(gq + 8) * 8 + tq * 2 + 1] += v3;
                    }
                }
            }
        }
        // only the consumer warps meet at the round's two barriers: the producer warp keeps filling the
        // ring with the next round's rows meanwhile
        if (consumer) asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers * 32) : "memory");   // partial sums are in the slots
        if (consumer && G > 0 && !u_ready) {   // u comes from the shrink kernel: fetched once into shared memory
            grid_dependency_wait();
            grid_launch_dependents();
            for (int i = tid; i < T * kRankPad / 4; i += kDecConsumers * 32)
                reinterpret_cast<float4*>(u_s)[i] = reinterpret_cast<const float4*>(u)[i];
            u_ready = true;
            asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers * 32) : "memory");
        }
        if (consumer && ok) {
            const bool lora = G > 0 && ctrl->bad_offsets == 0;
            const int per_token = nunits * kDecUnitRows;
            for (int e = tid; e < T * per_token; e += kDecConsumers * 32) {
                const int t = e / per_token, j = e % per_token;   // consecutive threads: consecutive n
                if (j >= round_rows) continue;
                const int un = j / kDecUnitRows, r = j % kDecUnitRows;
                const int n = round_begin + j;
                float v = 0.f;
#pragma unroll
                for (int w = 0; w < kDecConsumers; ++w) v += slots[(un * kDecConsumers + w) * kDecSlotFloats + t * 8 + r];
                const int slot = lora ? ctrl->slot_of_row[t] : -1;
                if (slot >= 0) {
                    const int r8 = ((int)snap.rank[slot] + 7) >> 3;
                    const uint4* bp = reinterpret_cast<const uint4*>(arenaB + ((size_t)slot * N + n) * kRankPad);
                    const float4* up = reinterpret_cast<const float4*>(u_s + t * kRankPad);
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
                y[(size_t)t * N + n] = __float2bfloat16_rn(v);
            }
        }
        if (consumer) asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers * 32) : "memory");   // slots are free for the next round
    }
    if (ctrl->abort) __nanosleep(50000);   // gave up: let copies still in flight land before the CTA goes away
    if (tid == 0 && ctrl->abort) atomicOr(status, LML_FLAG_TIMEOUT);
}

cudaError_t decode_init()
{
    // The shrink kernel asks for the same (maximal) shared-memory carve-out as the main kernel: an SM
    // cannot host CTAs of two kernels that want different L1 / shared-memory splits, and the main
    // kernel's CTAs must be able to start beside the shrink CTAs that are still running.
    cudaError_t e = cudaFuncSetAttribute(decode_shrink_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_main_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_main_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecSmemBytes);
}

cudaError_t launch_decode(const Arena& ar, const SlotSnapshot& snap, const DecodeArgs& a, cudaStream_t stream,
                          int* launches)
{
    const bool lora = a.G > 0;
    *launches = 0;
    if (lora) {
        int max_rank = 1;
        for (int i = 0; i < snap.max_slots; ++i) max_rank = snap.rank[i] > max_rank ? snap.rank[i] : max_rank;
        dim3 grid(a.T, (max_rank + 7) & ~7);   // one CTA per (position, j); the expand reads u in groups of 8 columns
        cudaLaunchConfig_t scfg = {};
        cudaLaunchAttribute sattr[1];
        pdl_config(scfg, sattr, grid, dim3(256), 0, stream);
        const __nv_bfloat16* arenaA = ar.A;
        uint32_t* sstatus = ar.status;
        const __nv_bfloat16* sx = (const __nv_bfloat16*)a.x;
        cudaError_t e = cudaLaunchKernelEx(&scfg, decode_shrink_kernel, snap, arenaA, sstatus, sx, a.T, a.d_in,
                                           a.seg_offsets, a.slot_ids, a.G, a.perm, a.u, a.row_slot);
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    const int row_pairs = (a.d_out + 1) / 2;   // at least two rows per CTA
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(row_pairs < a.num_sms ? row_pairs : a.num_sms);
    cfg.blockDim = dim3(kDecThreads);
    cfg.dynamicSmemBytes = kDecSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;   // with adapters the predecessor is the shrink kernel above, else the kernel waits at its top
    const __nv_bfloat16* xb = (const __nv_bfloat16*)a.x;
    const __nv_bfloat16* wb = (const __nv_bfloat16*)a.W0;
    __nv_bfloat16* yb = (__nv_bfloat16*)a.y;
    const float* up = a.u;
    const __nv_bfloat16* arenaB = ar.B;
    uint32_t* status = ar.status;
    const int32_t* so = a.seg_offsets;
    const int32_t* ids = a.slot_ids;
    const int32_t* pm = a.perm;
    cudaError_t e = a.T > 8 ? cudaLaunchKernelEx(&cfg, decode_main_kernel<true>, snap, arenaB, xb, wb, yb, up, so, ids, pm,
                                                 status, a.T, a.d_in, a.d_out, a.G)
                            : cudaLaunchKernelEx(&cfg, decode_main_kernel<false>, snap, arenaB, xb, wb, yb, up, so, ids, pm,
                                                 status, a.T, a.d_in, a.d_out, a.G);
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace lml
