// Decode path (T <= 16 tokens) for SEVERAL projections that read the same x (lora_mixed_linear_multi:
// q/k/v of an attention block): one launch, the LoRA shrink riding on the weight stream.
//
// The kernel is the persistent row-streaming design of lml_decode.cu (one CTA per SM, a producer warp
// feeding a ring of 8-row stages by bulk asynchronous copies, eight consumer warps with the x fragments
// in registers and mma.sync m16n8k16).  The rows of all projections' base weights form one virtual
// matrix that the grid shares out evenly (a CTA's range may cross from one projection into the next;
// units of eight rows never do); every projection has its own table, token binding and output.
//
// Where u = scale * x.A^T comes from differs from the single-projection kernel.  The live rows of A
// (every resident adapter's `rank` rows, all projections) are treated as further rows of the streamed
// matrix: they are cut into units of eight, dealt one to a CTA, and a CTA that holds such a unit runs it
// FIRST, through the same ring and the same MMAs as its rows of W0, before the kernel has even learnt
// which slot a token is bound to.  The unit's result is x.A_row^T for all tokens at once; a warp that is
// idle otherwise scales it, writes it to a small exchange buffer in global memory (u[live row][16 tokens],
// fp32) and counts it on a grid-wide counter.  Meanwhile the three further warps build the lookup tables,
// look the tokens' slots up, bring this CTA's rows of B into shared memory and, once the counter says that
// every live row has been published, collect the u values their tokens need.  The consumers never wait
// for that while rows still stream: the base sums of finished rounds wait in shared memory, and the
// expand is added when u is there (at the latest in the CTA's last round).  So the shrink costs no load
// of its own, needs no slot lookup before it starts, and its rows are fetched before the wait for the
// preceding work on the stream, exactly like W0 (the adapter arena is written only by register_adapter;
// the host runs the first such call after a registration with that early fetch switched off, and the
// kernel lets its own dependents start only after its wait, so that "before the preceding work" holds
// transitively).
//
// No CTA depends on the others being resident: a CTA whose peers have not published within a bounded
// time computes every live row itself, operands straight from global memory, with the same
// instruction sequence per row and hence the same bits.
// The kernel takes tables whose live rows are few (at most an eighth of the streamed rows, and at most
// kDsMaxLiveRows); the host sends everything else to the single-projection kernel, call by call.
#include <cstdlib>
#include <type_traits>

#include "lml_decode_common.cuh"
#include "lml_decode_stream.cuh"

namespace lml {

using namespace ptx;

constexpr int kDsConsumers = 8;
constexpr int kDsShrinkWarps = 3;
constexpr int kDsThreads = (kDsConsumers + 1 + kDsShrinkWarps) * 32;
constexpr int kDsUnitRows = 8;                   // rows per unit = the 8-wide MMA operand
constexpr int kDsSpan = 4096;                    // columns whose x fragments fit in registers (half of it for T > 8)
constexpr int kDsChunk = 2048;                   // columns per stage (one 4 KB bulk copy per row)
constexpr int kDsStepsPerChunk = kDsChunk / 32 / kDsConsumers;   // 8 k-steps per warp and stage
constexpr int kDsRowPitch = kDsChunk * 2 + 16;   // bytes; a quarter-warp's reads (2 rows x 4 lanes, 32 bytes apart) cover all banks
constexpr int kDsStageBytes = kDsUnitRows * kDsRowPitch;
constexpr int kDsStages = 4;
constexpr int kDsRoundUnits = 4;                 // units (<= 32 rows) reduced together
constexpr int kDsSlotFloats = 16 * kDsUnitRows;  // [token][row] partial sums of one warp for one unit
constexpr int kDsSlotBytes = kDsRoundUnits * kDsConsumers * kDsSlotFloats * 4;
constexpr int kDsUBytes = kDsMaxProj * 16 * kRankPad * 4;   // shared-memory copy of u, per projection
constexpr int kDsScratchBytes = kDsConsumers * kDsSlotFloats * 4;   // partial sums of the self-computed rows
constexpr int kDsSegCache = 128;                 // segments looked up in shared memory (single-projection segment form)
constexpr int kDsStageB = 10240;                 // staging of this CTA's rows of B, compact
constexpr int kDsDeferBytes = 12288;             // base sums of rounds that ended before u had arrived: 6 rounds of 16 x 32 or 12 of 8 x 32 fp32
constexpr int kDsDeferMax = 12;

struct DsLook {   // tables in shared memory
    DsProj proj[kDsMaxProj];
    int row0[kDsMaxProj + 1];                 // first virtual row of every projection, and the total
    int seg[kDsSegCache + 1];
    int ids[kDsSegCache];
    float scale_s[kDsMaxProj][kMaxSlots];
    uint8_t rank_s[kDsMaxProj][kMaxSlots];
    uint16_t live_end[kDsMaxProj * kMaxSlots];   // live rows up to and including (projection, slot), all projections in order
    int slot_of_row[kDsMaxProj][16];
    int rank_of_row[kDsMaxProj][16];
    int b_of_row[kDsMaxProj][16];     // byte offset in the staging buffer of the B block that serves (projection, token); -1: read global memory
    uint8_t b_lead[kDsMaxProj][16];   // the token is the first with its slot: it stands for the slot's block
    int cta_lo[kDsMaxProj];           // this CTA's rows of every projection: first virtual row ...
    int cta_rows[kDsMaxProj];         // ... and how many
    int def_start[kDsDeferMax][kDsRoundUnits];   // rounds whose sums wait in the buffer: first virtual row of each unit ...
    int def_nrows[kDsDeferMax][kDsRoundUnits];   // ... and its rows (0: no such unit)
    int def_nunits[kDsDeferMax];
    int u_complete;
    int u_seen;                       // one thread's look at the barrier below, shared so that every warp takes the same decision
    int bad_offsets;
};
struct DsCtrl {
    uint64_t full[kDsStages];
    uint64_t empty[kDsStages];
    uint64_t ufull;      // the three further warps have u, the slots and the copies of B in shared memory
    int abort;
};
constexpr int kDsLookBytes = (int)((sizeof(DsLook) + 15) & ~15u);
constexpr int kDsSmemBytes = 128 + kDsStages * kDsStageBytes + kDsSlotBytes + kDsUBytes + kDsScratchBytes + kDsStageB + kDsDeferBytes + 128 + kDsLookBytes;
static_assert(sizeof(DsCtrl) <= 128, "control block");
// 196 KB is the largest shared-memory carve-out that leaves the SM a useful L1 for the loads of x; the system keeps 1 KB per CTA
static_assert(kDsSmemBytes + 1024 <= 200704, "shared memory budget");

template <int kP> struct DsSnaps { SlotSnapshot s[kP]; };

// The virtual row space: projection q owns rows [row0[q], row0[q + 1]).
__device__ __forceinline__ int ds_proj_of(const DsLook* lk, int P, int row)
{
    int p = 0;
    for (int q = 1; q < P; ++q) if (row >= lk->row0[q]) p = q;
    return p;
}
// Next unit of a CTA's rows from `r` on: at most eight rows, never across a projection boundary.
__device__ __forceinline__ int ds_unit_rows(const int* row0, int P, int r, int end)
{
    int lim = min(end, r + kDsUnitRows);
#pragma unroll
    for (int q = 1; q < kDsMaxProj; ++q) { const int b = row0[q]; if (q < P && b > r && b < lim) lim = b; }
    return lim - r;
}
// The same from the kernel parameters (operands from the constant bank: no registers, no shared-memory table needed).
__device__ __forceinline__ int ds_unit_rows_prm(const DsParams& prm, int r, int end)
{
    int lim = min(end, r + kDsUnitRows), b = 0;
#pragma unroll
    for (int q = 0; q + 1 < kDsMaxProj; ++q) { b += prm.proj[q].N; if (q + 1 < prm.P && b > r && b < lim) lim = b; }
    return lim - r;
}
// Live row i -> (projection, slot, row j of the slot's A): the first table entry whose running count exceeds i.
__device__ __forceinline__ void ds_live_row(const DsLook* lk, int P, int i, int& p, int& slot, int& j)
{
    int lo = 0, hi = P * kMaxSlots - 1;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((int)lk->live_end[mid] > i) hi = mid; else lo = mid + 1;
    }
    p = lo / kMaxSlots;
    slot = lo % kMaxSlots;
    j = i - ((int)lk->live_end[lo] - (int)lk->rank_s[p][slot]);
}
// First live row of (projection, slot).
__device__ __forceinline__ int ds_live_first(const DsLook* lk, int p, int slot)
{
    return (int)lk->live_end[p * kMaxSlots + slot] - (int)lk->rank_s[p][slot];
}

// kTwo false: T <= 8, the second half of the 16-row MMA operand is zero and needs no registers.
// kMulti: the CTAs have more than one round of rows; the spans of d_in are then walked forwards and backwards in
//         turn, so that the x fragments a round ends with serve the next one without a reload.
// kP: how many table snapshots the launch carries (1, or kDsMaxProj for several projections).
template <bool kTwo, bool kMulti, int kP>
__global__ void __launch_bounds__(kDsThreads, 1) decode_stream_kernel(const __grid_constant__ DsSnaps<kP> snaps,
                                                                      const __grid_constant__ DsParams prm)
{
    extern __shared__ uint8_t ds_smem_raw[];
    const uint32_t raw = smem_u32(ds_smem_raw);
    const uint32_t ring = (raw + 127u) & ~127u;
    uint8_t* base_ptr = ds_smem_raw + (ring - raw);
    float* slots = reinterpret_cast<float*>(base_ptr + kDsStages * kDsStageBytes);            // [unit][warp][token][row]
    float* u_s = reinterpret_cast<float*>(base_ptr + kDsStages * kDsStageBytes + kDsSlotBytes);   // [projection][16][64]
    float* scratch = reinterpret_cast<float*>(base_ptr + kDsStages * kDsStageBytes + kDsSlotBytes + kDsUBytes);
    uint8_t* stage_b_s = base_ptr + kDsStages * kDsStageBytes + kDsSlotBytes + kDsUBytes + kDsScratchBytes;
    float* defer_s = reinterpret_cast<float*>(stage_b_s + kDsStageB);
    DsCtrl* ctrl = reinterpret_cast<DsCtrl*>(stage_b_s + kDsStageB + kDsDeferBytes);
    DsLook* lk = reinterpret_cast<DsLook*>(stage_b_s + kDsStageB + kDsDeferBytes + 128);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int P = prm.P, T = prm.T, K = prm.K;
    const bool lora = prm.live_rows > 0;            // the call has adapters to apply (G > 0 and live rows in the tables)
    const int L = prm.live_rows;
    const int n_au = (L + kDsUnitRows - 1) / kDsUnitRows;
    constexpr int kSpan = kTwo ? kDsSpan / 2 : kDsSpan;
    constexpr int kChunksPerSpan = kSpan / kDsChunk;
    const int nspans = (K + kSpan - 1) / kSpan;

    volatile int* abort = &ctrl->abort;
    const bool consumer = warp < kDsConsumers;
    const bool producer = warp == kDsConsumers;
    const bool shrinker = warp > kDsConsumers;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;

    // The producer warp sets the ring's barriers up, everybody meets once so that they are seen, and the producer
    // starts copying at once, with nothing but kernel parameters in hand; the tables that the other roles need are
    // built meanwhile (indexed reads of kernel parameters are slow the first time: they stay off the copy path).
    if (producer && lane == 0) {
        for (int s = 0; s < kDsStages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), kDsConsumers);
        }
        mbar_init(smem_u32(&ctrl->ufull), kDsShrinkWarps * 32);
        ctrl->abort = 0;
        fence_mbar_init();
    }
    asm volatile("bar.sync 4, %0;" ::"n"(kDsThreads) : "memory");   // the barriers are set up

    // this CTA's share: at most one unit of live rows of A, and a contiguous range of the virtual rows of W0 that
    // is the shorter for it, so that every CTA streams about the same number of bytes
    const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
    const int Ntot = prm.n_total;
    const int au_lo = (int)((long long)cta * n_au / grid), au_hi = (int)((long long)(cta + 1) * n_au / grid);
    const bool has_a = au_hi > au_lo;             // (the host launches only when n_au <= grid: one unit at most)
    const int a_rows = has_a ? min(kDsUnitRows, L - au_lo * kDsUnitRows) : 0;
    const int comp = (Ntot + kDsUnitRows * n_au) / grid >= 2 * kDsUnitRows ? kDsUnitRows : 0;
    const long long vtot = (long long)Ntot + (long long)comp * n_au;
    const int row_begin = (int)(vtot * cta / grid) - comp * au_lo;
    const int row_end = (int)(vtot * (cta + 1) / grid) - comp * au_hi;

    // ---- producer warp --------------------------------------------------------------------------------------------
    // W0 is the frozen base weight and the live rows of A belong to registrations that completed before the work
    // preceding this call (the host says so with early_adapters), so neither depends on that work; only the other
    // warps, which read x and the token bindings, wait for it.  Lane r copies this stage's 4 KB of row r.  The
    // warp never waits for a round's epilogue, only for free stages.
    if (producer) {
        // The stages go out in the order in which the consumers take them: position `pos` of that order uses slot
        // pos mod 4 of the ring.
        int pos = 0;
        auto put_stage = [&](int rows, const __nv_bfloat16* src, int cols) {   // src: this lane's row
            const int sl = pos % kDsStages;
            ok = ok && mbar_wait_warp(smem_u32(&ctrl->empty[sl]), (uint32_t)(((pos / kDsStages) & 1) ^ 1), abort);
            if (ok) {
                if (lane == 0) mbar_arrive_expect_tx(smem_u32(&ctrl->full[sl]), (uint32_t)(rows * cols * 2));
                __syncwarp();
                if (lane < rows)
                    bulk_copy_g2s(ring + sl * kDsStageBytes + lane * kDsRowPitch, src, (uint32_t)(cols * 2), smem_u32(&ctrl->full[sl]));
            }
            ++pos;
        };
        if (has_a) {
            // where the unit's rows live: live row i is row j of (projection, slot), counting the tables' ranks in order
            const int i = au_lo * kDsUnitRows + lane;   // lane r < a_rows looks for its own row
            const __nv_bfloat16* src = nullptr;
            int before = 0;
#pragma unroll
            for (int q = 0; q < kP; ++q) {
                if (q >= P) continue;
                const SlotSnapshot& sn = snaps.s[q];
                for (int sl = 0; sl < sn.max_slots; ++sl) {   // (uniform loop over at most 64 slots: every lane walks the same table)
                    const int rk = (int)sn.rank[sl];
                    if (lane < a_rows && i >= before && i < before + rk)
                        src = prm.proj[q].arenaA + ((size_t)sl * kRankPad + (i - before)) * K;
                    before += rk;
                }
            }
            if (!prm.early_adapters) grid_dependency_wait();   // a registration may be the very work before this call
            for (int sp = 0; sp < nspans && ok; ++sp) {   // the unit of A: spans forwards
                const int k_begin = sp * kSpan;
                const int span = min(kSpan, K - k_begin);
                const int nchunks = (span + kDsChunk - 1) / kDsChunk;
                for (int kc = 0; kc < nchunks && ok; ++kc)
                    put_stage(a_rows, src + k_begin + kc * kDsChunk, min(kDsChunk, span - kc * kDsChunk));
            }
        }
        int round = has_a ? 1 : 0;   // (parity of the span direction: the consumers count the same way)
        for (int r = row_begin; r < row_end && ok; ++round) {
            // the round's units: up to four, none across a projection boundary
            const int r_round = r;
            int nunits = 0;
            while (nunits < kDsRoundUnits && r < row_end) { r += ds_unit_rows_prm(prm, r, row_end); ++nunits; }
            const bool backwards = kMulti && (round & 1) != 0;
            for (int si = 0; si < nspans && ok; ++si) {
                const int sp = backwards ? nspans - 1 - si : si;
                const int k_begin = sp * kSpan;
                const int span = min(kSpan, K - k_begin);
                const int nchunks = (span + kDsChunk - 1) / kDsChunk;
                int rr = r_round;
#pragma unroll 1
                for (int un = 0; un < nunits && ok; ++un) {
                    const int rows = ds_unit_rows_prm(prm, rr, row_end);
                    // which projection's weight the unit belongs to
                    const __nv_bfloat16* w0p = prm.proj[0].W0;
                    int pr0 = 0, b = 0;
#pragma unroll
                    for (int q = 1; q < kDsMaxProj; ++q) {
                        b += prm.proj[q - 1].N;
                        if (q < P && rr >= b) { w0p = prm.proj[q].W0; pr0 = b; }
                    }
                    const __nv_bfloat16* src = w0p + (size_t)(rr - pr0 + lane) * K + k_begin;
                    for (int kc = 0; kc < nchunks && ok; ++kc)
                        put_stage(rows, src + kc * kDsChunk, min(kDsChunk, span - kc * kDsChunk));
                    rr += rows;
                }
            }
        }
    } else {
        grid_dependency_wait();     // launched as a programmatic dependent: the work before this call is complete now
        // Dependents may start only now: a kernel that follows this one fetches rows of A before its own wait,
        // and what it may rely on is that everything BEFORE its predecessor has completed.
        if (tid == 0) grid_launch_dependents();
    }

    // ---- tables for the epilogue and the lookup, built by the three further warps from the kernel parameters -----
    // (off the consumers' way to their loads of x: indexed reads of kernel parameters are slow the first time, and
    // slower still once the weight stream is running; the consumers pick the tables up before their first epilogue)
    if (shrinker) {
        const int sw = warp - kDsConsumers - 1;
        if (sw == 0) {
            if (lane < kDsMaxProj) lk->proj[lane] = prm.proj[lane < P ? lane : 0];
            if (lane == 0) {
                lk->bad_offsets = 0;
                lk->u_complete = 0;
                int r = 0;
                for (int q = 0; q < P; ++q) { lk->row0[q] = r; r += prm.proj[q].N; }
                for (int q = P; q <= kDsMaxProj; ++q) lk->row0[q] = r;
            }
            for (int i = lane; i < kDsMaxProj * 16; i += 32) {
                (&lk->slot_of_row[0][0])[i] = -1;
                (&lk->rank_of_row[0][0])[i] = 0;
                (&lk->b_of_row[0][0])[i] = -1;
                (&lk->b_lead[0][0])[i] = 0;
            }
        }
        if (sw == (kDsShrinkWarps > 2 ? 1 : 0)) {
#pragma unroll
            for (int q = 0; q < kP; ++q) {
                lk->scale_s[q][lane] = snaps.s[q].scale[lane];
                lk->scale_s[q][lane + 32] = snaps.s[q].scale[lane + 32];
            }
        }
        if (sw == kDsShrinkWarps - 1) {
            // ranks and the running count of live rows, projection after projection, slots in order
            int carry = 0;
#pragma unroll
            for (int q = 0; q < kP; ++q) {
                const SlotSnapshot& sn = snaps.s[q];
                const bool on = q < P && lora;
                const int r0 = (on && lane < sn.max_slots) ? (int)sn.rank[lane] : 0;
                const int r1 = (on && lane + 32 < sn.max_slots) ? (int)sn.rank[lane + 32] : 0;
                int i0 = r0, i1 = r1;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v0 = __shfl_up_sync(0xffffffffu, i0, o), v1 = __shfl_up_sync(0xffffffffu, i1, o);
                    if (lane >= o) { i0 += v0; i1 += v1; }
                }
                const int t0 = __shfl_sync(0xffffffffu, i0, 31), t1 = __shfl_sync(0xffffffffu, i1, 31);
                lk->rank_s[q][lane] = (uint8_t)r0;
                lk->rank_s[q][lane + 32] = (uint8_t)r1;
                lk->live_end[q * kMaxSlots + lane] = (uint16_t)(carry + i0);
                lk->live_end[q * kMaxSlots + lane + 32] = (uint16_t)(carry + t0 + i1);
                carry += t0 + t1;
            }
            for (int q = kP; q < kDsMaxProj; ++q) {   // (only so that the search over the whole table is defined)
                lk->rank_s[q][lane] = 0; lk->rank_s[q][lane + 32] = 0;
                lk->live_end[q * kMaxSlots + lane] = (uint16_t)carry; lk->live_end[q * kMaxSlots + lane + 32] = (uint16_t)carry;
            }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kDsShrinkWarps * 32) : "memory");   // these warps see the tables ...
        asm volatile("bar.arrive 5, %0;" ::"n"((kDsConsumers + kDsShrinkWarps) * 32) : "memory");   // ... and the consumers will
    }

    // ---- the three further warps: token bindings, this CTA's rows of B, and the u values of its tokens ----------
    if (shrinker && lora) {
        const int sw = warp - kDsConsumers - 1;
        const int me = tid - (kDsConsumers + 1) * 32;   // 0 .. 95
        if (sw == 0) {
            // The slot of every row of x, per projection.  Tokens form: one id per row and projection (all loads
            // issued before the first is used: one memory round trip).  Segments form (one projection): the
            // segment arrays go to shared memory and are searched there; calls with more segments than the cache
            // holds search global memory.
            const bool by_token = prm.proj[0].token_slots != nullptr;
            int slot_p[kP];
            int bad = 0, bad_perm = 0;
            unsigned bad_slot_mask = 0;   // bit q: projection q saw an id that names no live adapter
            if (by_token) {
                int id[kP];
#pragma unroll
                for (int q = 0; q < kP; ++q) id[q] = (q < P && lane < T) ? __ldg(lk->proj[q].token_slots + lane) : -1;
#pragma unroll
                for (int q = 0; q < kP; ++q) {
                    int s = id[q];
                    if (q < P && lane < T && lk->proj[q].adapter_map) s = resolve_adapter(snaps.s[q], lk->proj[q].adapter_map, s);
                    const bool live = s >= 0 && s < kMaxSlots && lk->rank_s[q][s] > 0;
                    if (q < P && lane < T && !live && s != -1) bad_slot_mask |= 1u << q;   // same rule as the segmentation pass
                    slot_p[q] = live ? s : -1;
                }
                if (lane < T) {
#pragma unroll
                    for (int q = 0; q < kP; ++q) if (q < P) lk->slot_of_row[q][lane] = slot_p[q];
                }
            } else {
                const int G = prm.G;
                const bool cached = G <= kDsSegCache;
                int my_row = lane;
                int so[kDsSegCache / 32 + 1], si[kDsSegCache / 32 + 1];
                if (cached) {
#pragma unroll
                    for (int i = 0; i <= kDsSegCache / 32; ++i) {
                        const int g = lane + 32 * i;
                        so[i] = g <= G ? __ldg(prm.seg_offsets + g) : 0;
                        si[i] = g < G ? __ldg(prm.slot_ids + g) : -1;
                    }
                }
                if (prm.perm && lane < T) my_row = __ldg(prm.perm + lane);
                if (cached) {
#pragma unroll
                    for (int i = 0; i <= kDsSegCache / 32; ++i) {
                        const int g = lane + 32 * i;
                        if (g <= G) lk->seg[g] = so[i];
                        if (g < G) lk->ids[g] = si[i];
                    }
                }
                __syncwarp();
                auto rank_of = [&](int sl) { return (sl >= 0 && sl < kMaxSlots) ? (int)lk->rank_s[0][sl] : 0; };
                int slot = -1, bad_slot = 0;
                const bool row_ok = lane < T && my_row >= 0 && my_row < T;
                if (cached) {
                    for (int g = lane; g < G; g += 32) {
                        const int s0 = lk->seg[g], s1 = lk->seg[g + 1], sl = lk->ids[g];
                        if (s1 < s0 || s0 < 0 || s1 > T) bad = 1;
                        if (sl != -1 && s1 > s0 && rank_of(sl) == 0) bad_slot = 1;   // an empty segment may name anything
                    }
                    if (lane == 0 && (lk->seg[0] != 0 || lk->seg[G] != T)) bad = 1;
                    if (row_ok) {   // first segment whose end lies beyond this position
                        int lo = 0, hi = G;
                        while (lo < hi) {
                            const int mid = (lo + hi) >> 1;
                            if (lk->seg[mid + 1] > lane) hi = mid; else lo = mid + 1;
                        }
                        if (lo < G && rank_of(lk->ids[lo]) > 0) slot = lk->ids[lo];
                    }
                } else {
                    for (int g = lane; g < G; g += 32) {
                        const int s0 = __ldg(prm.seg_offsets + g), s1 = __ldg(prm.seg_offsets + g + 1), sl = __ldg(prm.slot_ids + g);
                        if (s1 < s0 || s0 < 0 || s1 > T) bad = 1;
                        if (sl != -1 && s1 > s0 && rank_of(sl) == 0) bad_slot = 1;
                    }
                    if (lane == 0 && (__ldg(prm.seg_offsets) != 0 || __ldg(prm.seg_offsets + G) != T)) bad = 1;
                    if (row_ok) {
                        const int g = seg_upper(prm.seg_offsets, G, lane);
                        if (g < G) { const int sl = __ldg(prm.slot_ids + g); if (rank_of(sl) > 0) slot = sl; }
                    }
                }
                bad = __any_sync(0xffffffffu, bad);
                if (bad_slot) bad_slot_mask = 1u;
                if (!bad && lane < T) {
                    if (row_ok) lk->slot_of_row[0][my_row] = slot; else bad_perm = 1;
                }
            }
            bad_perm = __any_sync(0xffffffffu, bad_perm);
#pragma unroll
            for (int q = 0; q < kP; ++q) {
                const unsigned any_bad = __any_sync(0xffffffffu, (bad_slot_mask >> q) & 1u);
                if (q < P && lane == 0 && blockIdx.x == 0) {
                    const unsigned f = (any_bad ? LML_FLAG_BAD_SLOT : 0u) |
                                       (q == 0 ? ((bad ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_perm ? LML_FLAG_BAD_PERM : 0u)) : 0u);
                    if (f) atomicOr(lk->proj[q].status, f);
                }
            }
            if (lane == 0) lk->bad_offsets = bad;
            __syncwarp();
            // Per projection and row of x: the rank, and where the row's block of B goes in the staging buffer.  The
            // expand reads, per distinct slot, the first ceil(rank / 8) 16-byte chunks of this CTA's rows of B,
            // chunk-major ([chunk][row]: consecutive threads of the epilogue read consecutive 16 bytes); the first
            // row of x with a slot stands for the slot's block, blocks are laid out as long as they fit.
            int chunk_base = 0;
#pragma unroll
            for (int q = 0; q < kP; ++q) {
                if (q >= P) continue;
                const int lo = max(row_begin, lk->row0[q]), hi = min(row_end, lk->row0[q + 1]);
                const int rows_q = max(0, hi - lo);
                const int slot = lane < T ? lk->slot_of_row[q][lane] : -1;
                const int rank = slot >= 0 ? (int)lk->rank_s[q][slot] : 0;
                const unsigned same = __match_any_sync(0xffffffffu, slot);
                const int first = __ffs(same) - 1;
                const bool leader = rank > 0 && first == lane;
                const int chunks = leader ? rows_q * ((rank + 7) >> 3) : 0;
                int incl = chunks;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                const int fits = (chunk_base + incl) * 16 <= kDsStageB;
                const int my_off = __shfl_sync(0xffffffffu, fits ? (chunk_base + incl - chunks) * 16 : -1, first);
                if (lane < 16) {
                    lk->rank_of_row[q][lane] = rank;
                    lk->b_of_row[q][lane] = (rank > 0 && rows_q > 0) ? my_off : -1;
                    lk->b_lead[q][lane] = (leader && rows_q > 0) ? 1 : 0;
                }
                if (lane == 0) { lk->cta_lo[q] = lo; lk->cta_rows[q] = rows_q; }
                chunk_base += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        if (sw == 1 && has_a) {
            // the unit of A that this CTA's consumers have just multiplied: u[live row][token] = scale * sum of the
            // eight warps' partial sums (in warp order), written for the whole grid and counted with a release
            asm volatile("bar.sync 6, %0;" ::"n"(kDsConsumers * 32 + 32) : "memory");
            if (!ctrl->abort) {
#pragma unroll
                for (int k = 0; k < kDsSlotFloats / 32; ++k) {
                    const int e = lane + 32 * k, t = e >> 3, r = e & 7;
                    if (r < a_rows) {
                        float v = 0.f;
#pragma unroll
                        for (int w = 0; w < kDsConsumers; ++w) v += scratch[w * kDsSlotFloats + e];
                        int p, slot, j;
                        ds_live_row(lk, P, au_lo * kDsUnitRows + r, p, slot, j);
                        prm.u[(size_t)(au_lo * kDsUnitRows + r) * 16 + t] = v * lk->scale_s[p][slot];
                    }
                }
                __syncwarp();
                if (lane == 0) red_release_gpu_add(prm.sync_words, (unsigned)a_rows);
            }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kDsShrinkWarps * 32) : "memory");   // the slots are known
        // this CTA's rows of B into the staging buffer (16-byte asynchronous copies, all in flight at once);
        // blocks that did not fit are asked into L2 and read from there by the epilogue
        for (int q = 0; q < P; ++q) {
            const int rows_q = lk->cta_rows[q];
            const int N = lk->proj[q].N;
            const int n0 = lk->cta_lo[q] - lk->row0[q];
            for (int t = 0; t < T; ++t) {
                if (!lk->b_lead[q][t]) continue;
                const int rank = lk->rank_of_row[q][t], r8 = (rank + 7) >> 3;
                const bool compact = rank <= kRankCompact;   // 32-byte rows back to back instead of a quarter of a padded row each
                const int pitch = compact ? kRankCompact * 2 : kRankPad * 2;
                const char* b = compact ? reinterpret_cast<const char*>(lk->proj[q].arenaBc + ((size_t)lk->slot_of_row[q][t] * N + n0) * kRankCompact)
                                        : reinterpret_cast<const char*>(lk->proj[q].arenaB + ((size_t)lk->slot_of_row[q][t] * N + n0) * kRankPad);
                const int off = lk->b_of_row[q][t];
                if (off >= 0) {
                    for (int i = me; i < rows_q * r8; i += kDsShrinkWarps * 32) {
                        const int c = i / rows_q, r = i - c * rows_q;
                        cp_async_16(smem_u32(stage_b_s) + off + i * 16, b + (size_t)r * pitch + c * 16);
                    }
                } else {
                    for (int r = me; r < rows_q; r += kDsShrinkWarps * 32) prefetch_l2(b + (size_t)r * pitch);
                }
            }
        }
        // u in shared memory starts as zeros: the expand reads a row's columns up to the next multiple of eight
        for (int i = me; i < P * 16 * kRankPad / 4; i += kDsShrinkWarps * 32)
            reinterpret_cast<float4*>(u_s)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        // Wait until every live row has been published.  This CTA never depends on it: nothing guarantees that the
        // whole grid is resident at once (the launch is an ordinary one), so after a bounded wait the consumer
        // warps compute every row themselves, bit for bit the same, and the CTA makes room for the others.
        if (sw == 0 && lane == 0) {
            const long long t_wait = clock64();
            int complete = 1;
            while (ld_acquire_gpu(prm.sync_words) < (unsigned)L) {
                if (clock64() - t_wait > (long long)prm.patience) { complete = 0; break; }
            }
            lk->u_complete = complete;
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kDsShrinkWarps * 32) : "memory");
        if (lk->u_complete) {
            // the values this CTA's tokens need: u[live row of (slot, j)][token]; half a warp per (projection, token)
            // pair, 24 pairs per memory round trip
            const int half = lane >> 4, hl = lane & 15;
            for (int base = 0; base < P * 16; base += 8 * kDsShrinkWarps) {
                float v[4][4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int pair = base + (k * kDsShrinkWarps + sw) * 2 + half;
                    const int q = pair >> 4, t = pair & 15;
                    const int rank = pair < P * 16 ? lk->rank_of_row[q][t] : 0;
                    const float* src = prm.u + (size_t)(rank > 0 ? ds_live_first(lk, q, lk->slot_of_row[q][t]) : 0) * 16 + t;
#pragma unroll
                    for (int m = 0; m < 4; ++m) v[k][m] = hl + 16 * m < rank ? __ldcg(src + (hl + 16 * m) * 16) : 0.f;
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int pair = base + (k * kDsShrinkWarps + sw) * 2 + half;
                    const int rank = pair < P * 16 ? lk->rank_of_row[pair >> 4][pair & 15] : 0;
#pragma unroll
                    for (int m = 0; m < 4; ++m)
                        if (hl + 16 * m < rank) u_s[pair * kRankPad + hl + 16 * m] = v[k][m];
                }
            }
        }
        cp_async_wait_all();   // this thread's chunks of B have landed
        // tell the consumers that u_s, the slots, bad_offsets and the copies of B are final
        mbar_arrive(smem_u32(&ctrl->ufull));   // (the consumers can test this one without waiting)
    }

    // ---- consumer warps -----------------------------------------------------------------------------------------
    // Each warp owns a fixed slice of K (k-steps warp*8 .. warp*8+7 of every 2048-column chunk); its x fragments of
    // the current span stay in registers for every row that streams by.
    const int gq = lane >> 2, tq = lane & 3;
    uint4 xa[kChunksPerSpan * kDsStepsPerChunk], xc[kTwo ? kChunksPerSpan * kDsStepsPerChunk : 1];
    int span_loaded = -1;
    // The x fragments of span sp into registers.  Fragment i of a chunk holds the 8 columns warp*256 + (i/2)*64 + tq*16 +
    // (i&1)*8 ..: fragments 2j and 2j+1 of a lane are 32 consecutive bytes of its row, fetched by one 32-byte load, so a
    // warp's load covers whole 128-byte lines.  The weights are read with the same permutation on either route.
    const bool x_wide = ((reinterpret_cast<uintptr_t>(prm.x) | (uintptr_t)((size_t)K * 2)) & 31u) == 0;
    auto ensure_x = [&](int sp) {
        if (sp == span_loaded) return;
        span_loaded = sp;
        const int k_begin = sp * kSpan, span = min(kSpan, K - k_begin);
        const bool ta = gq < T, tb = gq + 8 < T;
#pragma unroll
        for (int i = 0; i < kChunksPerSpan * kDsStepsPerChunk; i += 2) {
            const int c = (i / kDsStepsPerChunk) * kDsChunk + (warp * kDsStepsPerChunk + i % kDsStepsPerChunk) * 32 + tq * 16;
            const __nv_bfloat16* pa = prm.x + (size_t)gq * K + k_begin + c;
            const __nv_bfloat16* pb = prm.x + (size_t)(gq + 8) * K + k_begin + c;
            if (x_wide && c + 16 <= span) {
                if (ta) ldg_nc_v8(pa, xa[i], xa[i + 1]); else xa[i] = xa[i + 1] = make_uint4(0, 0, 0, 0);
                if (kTwo) { if (tb) ldg_nc_v8(pb, xc[i], xc[i + 1]); else xc[i] = xc[i + 1] = make_uint4(0, 0, 0, 0); }
            } else {
                const bool l0 = c < span, l1 = c + 8 < span;
                xa[i] = (l0 && ta) ? ldg_nc_v4(pa) : make_uint4(0, 0, 0, 0);
                xa[i + 1] = (l1 && ta) ? ldg_nc_v4(pa + 8) : make_uint4(0, 0, 0, 0);
                if (kTwo) {
                    xc[i] = (l0 && tb) ? ldg_nc_v4(pb) : make_uint4(0, 0, 0, 0);
                    xc[i + 1] = (l1 && tb) ? ldg_nc_v4(pb + 8) : make_uint4(0, 0, 0, 0);
                }
            }
        }
    };
    // One unit (up to eight rows) times one span of x: this warp's partial sums [token][row] into `out` (set on the
    // unit's first span, added on the others).  Operands from the ring (kGlobal false: the stages arrive in the
    // producer's order) or straight from global memory (kGlobal true: `grow` is the row of this lane's group).
    // Either way the same MMAs run in the same order on the same values, so a row's sums do not depend on the route.
    auto run_unit = [&](auto global_tag, float* out, int rows, int sp, bool first_span, const __nv_bfloat16* grow) {
        constexpr bool kGlobal = decltype(global_tag)::value;
        const int k_begin = sp * kSpan, span = min(kSpan, K - k_begin);
        const int nchunks = (span + kDsChunk - 1) / kDsChunk;
        const bool rv = gq < rows;   // lanes whose row of the 8-wide operand is real
        float acc4[4][4];            // four independent accumulator chains keep several MMAs in flight per warp
#pragma unroll
        for (int a = 0; a < 4; ++a) acc4[a][0] = acc4[a][1] = acc4[a][2] = acc4[a][3] = 0.f;
#pragma unroll
        for (int kc = 0; kc < kChunksPerSpan; ++kc) {
            if (kc < nchunks && ok) {
                if (!kGlobal) ok = mbar_wait_warp(smem_u32(&ctrl->full[stage]), phase, abort);
                if (ok) {
                    const uint32_t wbase = ring + stage * kDsStageBytes + gq * kDsRowPitch + tq * 32 + warp * (kDsStepsPerChunk * 64);
                    uint4 w[kDsStepsPerChunk];
                    if (!kGlobal && rows == kDsUnitRows && span - kc * kDsChunk >= kDsChunk) {
                        // a full stage (all but the ragged edges): straight-line code, no predicates: all of the
                        // stage's operand reads first, then its MMAs
#pragma unroll
                        for (int i = 0; i < kDsStepsPerChunk; ++i)
                            w[i] = lds128(wbase + (uint32_t)((i >> 1) * 128 + (i & 1) * 16));
#pragma unroll
                        for (int i = 0; i < kDsStepsPerChunk; ++i) {
                            const uint4 a0 = xa[kc * kDsStepsPerChunk + i];
                            const uint4 a1 = kTwo ? xc[kc * kDsStepsPerChunk + i] : make_uint4(0, 0, 0, 0);
                            mma_bf16_16816(acc4[(2 * i) & 3], a0.x, a1.x, a0.y, a1.y, w[i].x, w[i].y);
                            mma_bf16_16816(acc4[(2 * i + 1) & 3], a0.z, a1.z, a0.w, a1.w, w[i].z, w[i].w);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < kDsStepsPerChunk; ++i) {
                            const int c0 = kc * kDsChunk + (warp * kDsStepsPerChunk + (i & ~1)) * 32;   // the pair's 64 columns start here
                            const int cl = c0 + tq * 16 + (i & 1) * 8;                                   // this lane's 8 columns
                            const bool lv = rv && cl < span;
                            if (kGlobal) w[i] = lv ? ldg_nc_v4(grow + k_begin + cl) : make_uint4(0, 0, 0, 0);
                            else w[i] = lv ? lds128(wbase + (uint32_t)((i >> 1) * 128 + (i & 1) * 16)) : make_uint4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int i = 0; i < kDsStepsPerChunk; ++i) {
                            const int c0 = kc * kDsChunk + (warp * kDsStepsPerChunk + (i & ~1)) * 32;
                            if (c0 < span) {   // uniform across the warp: all lanes issue the MMAs or none
                                const uint4 a0 = xa[kc * kDsStepsPerChunk + i];
                                const uint4 a1 = kTwo ? xc[kc * kDsStepsPerChunk + i] : make_uint4(0, 0, 0, 0);
                                mma_bf16_16816(acc4[(2 * i) & 3], a0.x, a1.x, a0.y, a1.y, w[i].x, w[i].y);
                                mma_bf16_16816(acc4[(2 * i + 1) & 3], a0.z, a1.z, a0.w, a1.w, w[i].z, w[i].w);
                            }
                        }
                    }
                    if (!kGlobal) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[stage]));
                        if (++stage == kDsStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
        // fragment: c0,c1 = (token gq, rows 2tq, 2tq+1); c2,c3 = (token gq+8, same rows)
        float vs[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) vs[a] = (acc4[0][a] + acc4[1][a]) + (acc4[2][a] + acc4[3][a]);
        if (first_span) {
            out[gq * 8 + tq * 2] = vs[0];       out[gq * 8 + tq * 2 + 1] = vs[1];
            out[(gq + 8) * 8 + tq * 2] = vs[2]; out[(gq + 8) * 8 + tq * 2 + 1] = vs[3];
        } else {
            out[gq * 8 + tq * 2] += vs[0];       out[gq * 8 + tq * 2 + 1] += vs[1];
            out[(gq + 8) * 8 + tq * 2] += vs[2]; out[(gq + 8) * 8 + tq * 2 + 1] += vs[3];
        }
    };
    using RingTag = std::integral_constant<bool, false>;
    using GlobalTag = std::integral_constant<bool, true>;

    // The rounds.  A CTA that holds a unit of A runs it first, as a round of its own: x.A_row^T for all tokens; the
    // warps' partial sums go to a warp that is idle otherwise, which adds them up, scales them and publishes them
    // for the whole grid, and the consumers move on to their rows of W0 at once.
    bool u_ready = false, tables_seen = false;
    int ndefer = 0;
    bool a_pending = consumer && has_a;
    int round = 0;
    for (int r = consumer ? row_begin : row_end; a_pending || r < row_end; ++round) {
        const bool a_round = a_pending;
        a_pending = false;
        // the round's units: up to four, none across a projection boundary (the producer forms the same ones)
        const int r_round = r;
        int nunits = a_round ? 1 : 0;
        while (!a_round && nunits < kDsRoundUnits && r < row_end) { r += ds_unit_rows_prm(prm, r, row_end); ++nunits; }
        const bool backwards = kMulti && !a_round && (round & 1) != 0;
        for (int si = 0; si < nspans; ++si) {
            const int sp = backwards ? nspans - 1 - si : si;
            ensure_x(sp);
            int rr = r_round;
#pragma unroll 1
            for (int un = 0; un < nunits; ++un) {
                const int rows = a_round ? a_rows : ds_unit_rows_prm(prm, rr, row_end);
                float* out = a_round ? scratch + warp * kDsSlotFloats : slots + (un * kDsConsumers + warp) * kDsSlotFloats;
                if (ok) run_unit(RingTag{}, out, rows, sp, si == 0, nullptr);
                rr += rows;
            }
        }
        if (a_round) {
            asm volatile("bar.arrive 6, %0;" ::"n"(kDsConsumers * 32 + 32) : "memory");
            continue;
        }
        if (tid == 0) {   // the round's units for the epilogue (and, if the round is put off, for the one that completes it)
            int rr = r_round;
            for (int un = 0; un < kDsRoundUnits; ++un) {
                const int rows = un < nunits ? ds_unit_rows_prm(prm, rr, row_end) : 0;
                lk->def_start[ndefer][un] = rr; lk->def_nrows[ndefer][un] = rows;
                rr += rows;
            }
            lk->def_nunits[ndefer] = nunits;
        }
        if (tid == 0 && lora && !u_ready) lk->u_seen = mbar_test_wait(smem_u32(&ctrl->ufull), 0u) ? 1 : 0;
        // only the consumer warps meet at the round's two barriers: the producer keeps filling the ring meanwhile
        asm volatile("bar.sync 1, %0;" ::"n"(kDsConsumers * 32) : "memory");   // partial sums are in the slots
        if (!tables_seen) {   // first epilogue: the tables the other warps built
            asm volatile("bar.sync 5, %0;" ::"n"((kDsConsumers + kDsShrinkWarps) * 32) : "memory");
            tables_seen = true;
        }
        // The expand needs u, which the whole grid computes and which arrives some microseconds into the call.  The
        // consumers do not wait for it: until it is there, every thread keeps the base sums of its elements of the
        // finished rounds in shared memory (the same thread completes them later); only the last round, or a full
        // buffer, waits.  Every warp takes the same decision (one thread looked, before the barrier above).
        constexpr int kDefStride = kTwo ? 512 : 256;                  // elements of a round: 16 x 32 or 8 x 32
        constexpr int kDefRounds = kDsDeferBytes / (kDefStride * 4);
        static_assert(kDefRounds <= kDsDeferMax, "deferred rounds");
        if (lora && !u_ready) {
            bool seen = lk->u_seen != 0;
            if (!seen && (r >= row_end || ndefer == kDefRounds - 1)) {   // (the last free place is this round's own)
                int there = 1;
                if (lane == 0) there = mbar_wait_spin(smem_u32(&ctrl->ufull), 0u, abort) ? 1 : 0;
                seen = __shfl_sync(0xffffffffu, there, 0) != 0;
                if (!seen) ok = false;
            }
            u_ready = seen;
            if (u_ready && !lk->u_complete) {   // (the same verdict in every warp: they meet at barriers inside)
                // The peers' rows did not arrive in time: compute every live row here, operands from global memory.
                for (int a = 0; a < n_au; ++a) {
                    const int rows = min(kDsUnitRows, L - a * kDsUnitRows);
                    const __nv_bfloat16* grow = nullptr;
                    if (gq < rows) {
                        int p, slot, j;
                        ds_live_row(lk, P, a * kDsUnitRows + gq, p, slot, j);
                        grow = lk->proj[p].arenaA + ((size_t)slot * kRankPad + j) * K;
                    }
                    for (int sp = 0; sp < nspans; ++sp) {
                        ensure_x(sp);
                        run_unit(GlobalTag{}, scratch + warp * kDsSlotFloats, rows, sp, sp == 0, grow);
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kDsConsumers * 32) : "memory");
                    if (tid < kDsSlotFloats) {
                        const int t = tid >> 3, rr = tid & 7;
                        if (rr < rows && t < T) {
                            float v = 0.f;
#pragma unroll
                            for (int w = 0; w < kDsConsumers; ++w) v += scratch[w * kDsSlotFloats + tid];
                            int p, slot, j;
                            ds_live_row(lk, P, a * kDsUnitRows + rr, p, slot, j);
                            if (lk->slot_of_row[p][t] == slot) u_s[(p * 16 + t) * kRankPad + j] = v * lk->scale_s[p][slot];
                        }
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kDsConsumers * 32) : "memory");
                }
            }
        }
        if (ok) {
            const bool use_lora = lora && lk->bad_offsets == 0;
            // y[t][n] = base sum + u_t . B_slot[n] (the first ceil(rank / 8) chunks of the row), rounded once
            auto finish = [&](int t, int p, int n, float v) {
                const DsProj& pj = lk->proj[p];
                const int slot = use_lora ? lk->slot_of_row[p][t] : -1;
                if (slot >= 0) {
                    const int rank = lk->rank_of_row[p][t], r8 = (rank + 7) >> 3;
                    const int rows_cta = lk->cta_rows[p];
                    const uint4* bp = rank <= kRankCompact ? reinterpret_cast<const uint4*>(pj.arenaBc + ((size_t)slot * pj.N + n) * kRankCompact)
                                                           : reinterpret_cast<const uint4*>(pj.arenaB + ((size_t)slot * pj.N + n) * kRankPad);
                    const int bb = lk->b_of_row[p][t];
                    const uint4* bs = reinterpret_cast<const uint4*>(stage_b_s + bb) + (n - (lk->cta_lo[p] - lk->row0[p]));
                    const float4* up = reinterpret_cast<const float4*>(u_s + (p * 16 + t) * kRankPad);
                    float d = 0.f;
                    auto fma8 = [&](const uint4& b, int c) {
                        const float4 u0v = up[2 * c], u1v = up[2 * c + 1];
                        d = fmaf(u0v.x, bf16_lo(b.x), d); d = fmaf(u0v.y, bf16_hi(b.x), d);
                        d = fmaf(u0v.z, bf16_lo(b.y), d); d = fmaf(u0v.w, bf16_hi(b.y), d);
                        d = fmaf(u1v.x, bf16_lo(b.z), d); d = fmaf(u1v.y, bf16_hi(b.z), d);
                        d = fmaf(u1v.z, bf16_lo(b.w), d); d = fmaf(u1v.w, bf16_hi(b.w), d);
                    };
                    if (bb >= 0) {   // (two loops: with a select inside one loop the global loads no longer overlap)
                        for (int c = 0; c < r8; ++c) fma8(bs[c * rows_cta], c);
                    } else {
                        for (int c = 0; c < r8; ++c) fma8(ldg_nc_v4(bp + c), c);
                    }
                    v += d;
                }
                pj.y[(size_t)t * pj.N + n] = __float2bfloat16_rn(v);
            };
            // Every round's base sums go through the buffer of put-off rounds (each thread keeps its own elements);
            // whatever is in there is completed as soon as u is at hand: at once in a call without adapters.
            const int per_token = nunits * kDsUnitRows;
            for (int e = tid; e < T * per_token; e += kDsConsumers * 32) {
                const int t = e / per_token, j = e % per_token;   // consecutive threads: consecutive rows of W0
                const int un = j / kDsUnitRows, rr = j % kDsUnitRows;
                float v = 0.f;
#pragma unroll
                for (int w = 0; w < kDsConsumers; ++w) v += slots[(un * kDsConsumers + w) * kDsSlotFloats + t * 8 + rr];
                defer_s[ndefer * kDefStride + e] = v;   // read back by this very thread
            }
            ++ndefer;
            if (!lora || u_ready) {
                for (int dd = 0; dd < ndefer; ++dd) {
                    const int pt = lk->def_nunits[dd] * kDsUnitRows;
                    for (int e = tid; e < T * pt; e += kDsConsumers * 32) {
                        const int t = e / pt, j = e % pt;
                        const int un = j / kDsUnitRows, rr = j % kDsUnitRows;
                        if (rr >= lk->def_nrows[dd][un]) continue;
                        const int nv = lk->def_start[dd][un] + rr;
                        const int p = ds_proj_of(lk, P, nv);
                        finish(t, p, nv - lk->row0[p], defer_s[dd * kDefStride + e]);
                    }
                }
                ndefer = 0;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kDsConsumers * 32) : "memory");   // slots are free for the next round
    }
    if (ctrl->abort) __nanosleep(50000);   // gave up: let copies still in flight land before the CTA goes away
    if (tid == 0) {
        if (ctrl->abort) atomicOr(prm.proj[0].status, LML_FLAG_TIMEOUT);
        // Every CTA signs off when it is done (its rows of u are published, its own copy is taken); the last one
        // puts both counters back to zero for the next call.
        if (lora) {
            __threadfence();
            if (atomicAdd(prm.sync_words + 1, 1u) == gridDim.x - 1) {
                prm.sync_words[0] = 0u;
                prm.sync_words[1] = 0u;
            }
        }
    }
}

// ---- host side ------------------------------------------------------------------------------------------------

static int ds_grid(int n_total, int num_sms)
{
    const int row_pairs = (n_total + 1) / 2;   // at least two rows per CTA
    return row_pairs < num_sms ? row_pairs : num_sms;
}

static int ds_live_rows(const SlotSnapshot* snaps, int P)
{
    int live = 0;
    for (int q = 0; q < P; ++q)
        for (int i = 0; i < snaps[q].max_slots && i < kMaxSlots; ++i) live += snaps[q].rank[i];
    return live;
}

bool decode_stream_eligible(const SlotSnapshot* snaps, const int* d_out, int P, int /*d_in*/, bool has_adapters, int num_sms)
{
    if (P < 1 || P > kDsMaxProj) return false;
    long long n_total = 0;
    for (int q = 0; q < P; ++q) n_total += d_out[q];
    if (n_total > (1ll << 30)) return false;
    if (!has_adapters) return true;
    const int live = ds_live_rows(snaps, P);
    // streaming every live row must stay a small extra on top of W0, and one unit per CTA at most
    return live <= kDsMaxLiveRows && (long long)live * 8 <= n_total &&
           (live + kDsUnitRows - 1) / kDsUnitRows <= ds_grid((int)n_total, num_sms);
}

cudaError_t decode_stream_init()
{
    cudaError_t e = cudaSuccess;
    auto set = [&](auto kernel) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDsSmemBytes);
    };
    set(decode_stream_kernel<false, false, 1>); set(decode_stream_kernel<false, true, 1>);
    set(decode_stream_kernel<true, false, 1>);  set(decode_stream_kernel<true, true, 1>);
    set(decode_stream_kernel<false, false, kDsMaxProj>); set(decode_stream_kernel<false, true, kDsMaxProj>);
    set(decode_stream_kernel<true, false, kDsMaxProj>);  set(decode_stream_kernel<true, true, kDsMaxProj>);
    return e;
}

cudaError_t launch_decode_stream(const SlotSnapshot* snaps, DsParams prm, int num_sms, cudaStream_t stream)
{
    int n_total = 0;
    for (int q = 0; q < prm.P; ++q) n_total += prm.proj[q].N;
    for (int q = prm.P; q < kDsMaxProj; ++q) prm.proj[q] = prm.proj[0];
    prm.live_rows = prm.G > 0 ? ds_live_rows(snaps, prm.P) : 0;
    prm.n_total = n_total;
    const int grid = ds_grid(n_total, num_sms);
    const int n_au = (prm.live_rows + kDsUnitRows - 1) / kDsUnitRows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kDsThreads);
    cfg.dynamicSmemBytes = kDsSmemBytes;
    cfg.stream = stream;
    // An ordinary launch, as a programmatic dependent of whatever precedes it on the stream (the kernel waits
    // for that work itself, after it has started on W0 and A).  No CTA depends on the others being resident.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int rows_per_cta = (n_total + kDsUnitRows * n_au + grid - 1) / grid;
    const bool multi = rows_per_cta > kDsRoundUnits * kDsUnitRows;
    const bool two = prm.T > 8;
    if (prm.P == 1) {
        DsSnaps<1> sn;
        sn.s[0] = snaps[0];
        auto launch = [&](auto kernel) { return cudaLaunchKernelEx(&cfg, kernel, sn, prm); };
        if (two) return multi ? launch(decode_stream_kernel<true, true, 1>) : launch(decode_stream_kernel<true, false, 1>);
        return multi ? launch(decode_stream_kernel<false, true, 1>) : launch(decode_stream_kernel<false, false, 1>);
    }
    DsSnaps<kDsMaxProj> sn = {};
    for (int q = 0; q < prm.P; ++q) sn.s[q] = snaps[q];
    auto launch = [&](auto kernel) { return cudaLaunchKernelEx(&cfg, kernel, sn, prm); };
    if (two) return multi ? launch(decode_stream_kernel<true, true, kDsMaxProj>) : launch(decode_stream_kernel<true, false, kDsMaxProj>);
    return multi ? launch(decode_stream_kernel<false, true, kDsMaxProj>) : launch(decode_stream_kernel<false, false, kDsMaxProj>);
}


}  // namespace lml
