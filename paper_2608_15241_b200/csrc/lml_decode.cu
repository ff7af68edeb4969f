// Decode path (T <= 16 tokens): bandwidth-bound.  W0 is read exactly once.
//
// One kernel, decode_main_kernel: one persistent CTA per SM, each owning a contiguous, balanced
// range of W0 rows (N/148 of them, +-1), because an SM cannot take in much more than its fair share
// of HBM bandwidth and contiguous addresses stream best.  Twelve warps in three roles:
//   producer (1 warp)   copies 8 rows x 2048 columns per stage (one 4 KB bulk asynchronous copy per
//                       row) into a shared-memory ring, unit after unit, so the CTA walks its rows
//                       front to back; it runs ahead across rounds.  It starts right at kernel entry,
//                       before the wait for the preceding work on the stream (W0 does not depend on
//                       it), so HBM already streams this call's weights while that work drains.
//   consumers (8 warps) each own a fixed slice of K: their x fragments are loaded once into
//                       registers and reused for every row.  y^T += W0.x^T runs on mma.sync m16n8k16
//                       with the tokens as the 16-row operand (T <= 16 is exactly one tile; T <= 8
//                       uses a variant that feeds zeros for the upper half and keeps twice the span
//                       of x in registers) and 8 rows of W0 as the 8-wide operand.  The k order
//                       inside a 32-wide step is permuted identically for both operands, which a dot
//                       product does not see, so operands are plain 16-byte loads.  Per-warp partial
//                       sums go to per-warp slots and are added in a fixed order; the LoRA expand
//                       sum_j u[t][j] B_s[n][j] is added in fp32 before the single bf16 rounding.
//   shrink (3 warps)    only when the call has adapters: look up each row's slot (from segments, cached in
//                       shared memory, or from one slot id per row), then compute this CTA's share of
//                       u[row][j] = scale_s * sum_k x[row][k] A_s[j][k] (fp32).  The dot products are dealt
//                       out over the whole grid in groups of 1, 2 or 4 columns of one row; a group's
//                       operands are all in flight at once, in registers (one memory round trip per
//                       4608 columns).  This CTA's rows of B of the slots that the call names come
//                       into shared memory meanwhile (rank <= 16: one bulk copy per slot, issued by
//                       the lookup warp).  Each result goes to
//                       the table's exchange block as one 64-bit word, the value beside this launch's
//                       mark, followed by a plain add on a grid-wide counter (no fence anywhere); the
//                       warps wait for the counter, then read the entries, taking only those that carry
//                       the mark, and stage all of u in shared memory.  When the table's live
//                       adapters are very few, their rows of A are asked into L2 at kernel entry, ahead of
//                       the weight stream.  The consumers meet the shrink warps once, at their first
//                       epilogue.  No CTA depends on the others being resident: after a bounded wait
//                       for their shares it computes all of u itself (same arithmetic, same bits).  So
//                       the launch is an ordinary one and needs no co-residency guarantee.
// d_in wider than a span is walked span by span.  All waits are bounded.
// Several projections that read the same x (q / k / v, gate / up, or the two bindings of a dual-version call over
// one W0) run as one launch: the grid is dealt out over the projections in proportion to their rows, and a CTA
// works on its projection as if that were the whole call, so the results are those of separate calls bit for bit
// and the fixed costs of a call (the wait for the preceding work, the fetch of x, the tail) are paid once.
// CTAs with more than one round of 32 rows (wide layers) come in two further builds of the kernel: the
// spans are walked forwards and backwards in turn, so that the x fragments a round ends with serve the
// next one without a reload; and, with adapters, the expand of early rounds is put off until u has
// arrived (the base sums wait in shared memory), so only a CTA's last round can wait for the grid.  The
// expand's operand B is staged compactly (the chunks a row really has) for all of a CTA's rows at once.
#include <cstdlib>
#include "lml_internal.cuh"
#include "lml_ptx_sm100.cuh"
#include <type_traits>

#include "lml_decode_common.cuh"

namespace lml {

using namespace ptx;

constexpr int kDecMaxTables = LML_MAX_PROJECTIONS;   // tables (projections proper) that one launch can serve
constexpr int kDecMaxProj = kDecMaxBlocks;           // parts of a launch: projections, bindings of a dual call, blocks of 16 tokens
constexpr int kDecConsumers = 8;                 // consumer warps
constexpr int kDecShrinkWarps = 3;               // warps after the producer warp: the LoRA shrink
constexpr int kDecThreads = (kDecConsumers + 1 + kDecShrinkWarps) * 32;
constexpr int kDecUnitRows = 8;                  // W0 rows per unit = the 8-wide MMA operand
constexpr int kDecSpan = 4096;                   // columns whose x fragments fit in registers (half of it for T > 8)
constexpr int kDecChunk = 2048;                  // columns per stage (one 4 KB bulk copy per row)
constexpr int kDecChunksPerSpan = kDecSpan / kDecChunk;             // 4
constexpr int kDecStepsPerChunk = kDecChunk / 32 / kDecConsumers;   // 8 k-steps per warp and stage
constexpr int kDecRowPitch = kDecChunk * 2 + 16; // bytes; one 16-byte chunk more than a multiple of 128: a quarter-warp's reads (2 rows x 4 lanes, 32 bytes apart) cover all banks
constexpr int kDecStageBytes = kDecUnitRows * kDecRowPitch;
constexpr int kDecStages = 4;                    // ring stages of a call with adapters
constexpr int kDecStagesBase = 5;                // of a call without any (see DecCfg)
constexpr int kDecRoundUnits = 4;                // units (= 32 rows) reduced together
constexpr int kDecSlotFloats = 16 * kDecUnitRows;   // [token][row] partial sums of one warp for one unit
constexpr int kDecSlotBytes = kDecRoundUnits * kDecConsumers * kDecSlotFloats * 4;
constexpr int kDecUBytes = 16 * kRankPad * 4;     // shared-memory copy of u for the epilogue
constexpr int kDecSegCache = 128;                 // segments whose offsets and slots are looked up in shared memory
constexpr int kDecDotGroup = 4;                    // dot products of one row of x that a CTA takes together
constexpr int kDecDotBytes = 40960;                // staging buffer: this CTA's rows of B of the slots that the call names
struct DecLookup {   // what the shrink warps work out about the call, in shared memory
    int seg[kDecSegCache + 1];
    int ids[kDecSegCache];
    float scale_s[kMaxSlots];
    uint8_t rank_s[kMaxSlots];
    int dot_end[16];        // running total of dot products up to and including each row of x
    int rank_of_row[16];
    float dot_part[kDecDotGroup][4];
    int u_complete;
    unsigned epoch;         // this launch's mark on the entries of u
    int pad[3];
    // what the expand needs to know about a row of x, in one word: bit 31 the row has an adapter; bits 0-7 its slot;
    // bits 8-11 ceil(rank / 8); bit 12 rank <= 16 (the compact arena serves it); bit 13 its block of B is in the staging
    // buffer, at 16 x bits 16-27 bytes
    unsigned row_info[16];
};
constexpr int kDecSegBytes = (int)sizeof(DecLookup);
constexpr int kDecDeferBytes = 2048;   // base sums of rounds whose expand is put off: 16 x 32 or 2 x (8 x 32) fp32
constexpr int kDecCtrlBytes = 320;
// A call without any adapter (G == 0) has no use for the staging buffer of B and takes a fifth ring stage instead: the
// deeper ring is worth 0.5 us on a 4096 x 4096 layer (8.24 -> 7.73 us).  With adapters a fifth stage loses (8.63 against
// 8.39 us even where the blocks of B still fit): the shrink warps' cold loads queue up behind whatever the ring has asked for.
// The third build lies between the two: five stages and what is left of the carve-out, 10.5 KB, as staging buffer, for
// calls whose blocks of B are sure to fit in that (few tokens or few rows per CTA; the launcher works out the worst
// case from the table's ranks): 8.20 -> 8.07 us on decode_q_proj.  Where the blocks do not fit, the fifth stage costs
// more than it brings (9.4 -> 10.4 us at 16 tokens and 11 slots), hence the choice per call.
constexpr int kDecVarFull = 0, kDecVarBase = 1, kDecVarSmall = 2;
constexpr int kDecDotBytesSmall = 10496;
template <int kVar> struct DecCfg {
    static constexpr int kStages = kVar == kDecVarFull ? kDecStages : kDecStagesBase;
    static constexpr int kDotBytes = kVar == kDecVarFull ? kDecDotBytes : (kVar == kDecVarBase ? 0 : kDecDotBytesSmall);
    static constexpr int kSmemBytes = 128 + kStages * kDecStageBytes + kDecSlotBytes + kDecUBytes + kDecCtrlBytes + kDecSegBytes + 8 + kDotBytes + kDecDeferBytes;
};
constexpr int kDecSmemBytes = DecCfg<kDecVarFull>::kSmemBytes;
// 196 KB is also the largest shared-memory carve-out that leaves the SM a useful L1 for the loads of x:
// one step more and the base-only call is 0.8 us slower.
static_assert(kDecSmemBytes + 1024 <= 200704 && DecCfg<kDecVarBase>::kSmemBytes + 1024 <= 200704 &&
              DecCfg<kDecVarSmall>::kSmemBytes + 1024 <= 200704 && kDecDotBytesSmall % 16 == 0, "shared memory budget");   // the system keeps 1 KB per CTA for itself

struct DecCtrl {
    uint64_t full[kDecStagesBase];
    uint64_t empty[kDecStagesBase];
    uint64_t ufull;      // the shrink warps' results (u, the slots, the copies of B) are in shared memory
    uint64_t bfull;      // the bulk copies of B (whole rows of the compact arena) have landed
    int abort;
    int bad_offsets;
    int slot_of_row[16];
    int b_of_row[16];    // byte offset, in the staging buffer, of the B copy that serves this row of x; -1: read B from global memory
    uint8_t b_lead[16];  // 1: this row of x is the first with its slot (it stands for the slot's block of B)
    uint8_t b_rows[16];  // 1: the block holds whole 32-byte rows of the compact arena, row after row (one bulk copy); 0: 16-byte chunks, chunk-major
};
static_assert(sizeof(DecCtrl) <= kDecCtrlBytes && kDecStagesBase >= kDecStages && (kDecSegBytes + 8) % 16 == 0, "control block");

// kTwo false: T <= 8, the second half of the 16-row MMA operand is zero and needs no registers.
// kMulti: the CTAs have more than one round of rows; compiled with the code that saves reloads of x between rounds.
// kPutOff: compiled with the code that puts the expand of early rounds off (kMulti calls with adapters).
// One projection of a launch: its table, base weight, binding and output, and the CTAs that work on it.
struct DecProj {
    const __nv_bfloat16* arenaA;
    const __nv_bfloat16* arenaB;
    const __nv_bfloat16* arenaBc;
    const __nv_bfloat16* W0;
    __nv_bfloat16* y;
    unsigned long long* u;      // this part's exchange block: [16][kRankPad] entries (value | mark << 32), then its three words
    const int32_t* seg_offsets;
    const int32_t* slot_ids;
    const int32_t* perm;
    const int32_t* token_slots;
    const int32_t* adapter_map;
    uint32_t* status;
    unsigned int* sync_words;   // the block's words: [0] the mark of the last launch that finished, [1] CTAs that have left, [2] entries written
    int N, G;
    int cta_begin, cta_count;   // CTAs [cta_begin, cta_begin + cta_count) of the grid
    // (what launches of several parts need comes last: the single-part build is sensitive to the layout of the fields above,
    // 0.25 us per call on a 4096 x 4096 layer were measured between two orders)
    const __nv_bfloat16* x;     // this part's rows of x ...
    int T;                      // ... and how many (<= 16)
    int snap_idx;               // its table's snapshot in the launch's list
};
// kP projections that read the same x (kP = 1: the plain call).  With several, the grid is dealt out over the
// projections in proportion to their rows; a CTA works on one projection as if that were the whole call (its own
// rows, its own share of that table's dot products, that table's counters), so one launch pays the fixed costs of a
// call (the wait for the preceding work, the fetch of x, the tail) once for all of them.
template <int kP> struct DecLaunch {
    SlotSnapshot snap[kP == 1 ? 1 : kDecMaxTables];
    DecProj proj[kP];
    const __nv_bfloat16* x;   // (kP == 1: the call's x and token count, as proj[0] has them)
    int T, K, P, patience;
};

template <bool kTwo, bool kMulti, bool kPutOff, int kP = 1, int kVar = kDecVarFull>
__global__ void __launch_bounds__(kDecThreads, 1) decode_main_kernel(const __grid_constant__ DecLaunch<kP> prm)
{
    int pi = 0;
    if (kP > 1)
        while (pi + 1 < prm.P && (int)blockIdx.x >= prm.proj[pi + 1].cta_begin) ++pi;
    const DecProj& pj = prm.proj[pi];
    const SlotSnapshot& snap = prm.snap[kP == 1 ? 0 : pj.snap_idx];
    const int cta = (int)blockIdx.x - pj.cta_begin, ncta = pj.cta_count;   // this CTA among those of its projection
    const __nv_bfloat16* __restrict__ arenaA = pj.arenaA;
    const __nv_bfloat16* __restrict__ arenaB = pj.arenaB;
    const __nv_bfloat16* __restrict__ arenaBc = pj.arenaBc;
    const __nv_bfloat16* __restrict__ x = kP == 1 ? prm.x : pj.x;
    const __nv_bfloat16* __restrict__ W0 = pj.W0;
    __nv_bfloat16* __restrict__ y = pj.y;
    unsigned long long* u = pj.u;
    const int32_t* __restrict__ seg_offsets = pj.seg_offsets;
    const int32_t* __restrict__ slot_ids = pj.slot_ids;
    const int32_t* __restrict__ perm = pj.perm;
    const int32_t* __restrict__ token_slots = pj.token_slots;
    const int32_t* __restrict__ adapter_map = pj.adapter_map;
    uint32_t* status = pj.status;
    constexpr bool kBase = kVar == kDecVarBase;
    constexpr int kS = DecCfg<kVar>::kStages, kDotBytes = DecCfg<kVar>::kDotBytes;
    const int T = kP == 1 ? prm.T : pj.T, K = prm.K, N = pj.N, G = kBase ? 0 : pj.G, patience = prm.patience;
    extern __shared__ uint8_t dec_smem_raw[];
    const uint32_t raw = smem_u32(dec_smem_raw);
    const uint32_t ring = (raw + 127u) & ~127u;
    uint8_t* base_ptr = dec_smem_raw + (ring - raw);
    float* slots = reinterpret_cast<float*>(base_ptr + kS * kDecStageBytes);   // [stage][warp][token][row]
    float* u_s = reinterpret_cast<float*>(base_ptr + kS * kDecStageBytes + kDecSlotBytes);   // [16][64]
    DecCtrl* ctrl = reinterpret_cast<DecCtrl*>(base_ptr + kS * kDecStageBytes + kDecSlotBytes + kDecUBytes);
    DecLookup* lk = reinterpret_cast<DecLookup*>(base_ptr + kS * kDecStageBytes + kDecSlotBytes + kDecUBytes + kDecCtrlBytes);
    uint8_t* dot_s = base_ptr + kS * kDecStageBytes + kDecSlotBytes + kDecUBytes + kDecCtrlBytes + kDecSegBytes + 8;   // 16-byte aligned
    float* defer_s = reinterpret_cast<float*>(dot_s + kDotBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // this CTA's rows: a contiguous, balanced range
    const int row_begin = (int)((long long)cta * N / ncta);
    const int row_end = (int)((long long)(cta + 1) * N / ncta);
    // x fragments of a span live in registers; with two 8-token blocks a span is half as wide, so
    // both variants hold 64 fragment registers and stay clear of spills
    constexpr int kSpan = kTwo ? kDecSpan / 2 : kDecSpan;
    constexpr int kChunksPerSpan = kSpan / kDecChunk;
    const int nspans = (K + kSpan - 1) / kSpan;

    volatile int* abort = &ctrl->abort;
    const bool consumer = warp < kDecConsumers;
    const bool producer = warp == kDecConsumers;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;

    // ---- producer warp ----------------------------------------------------------------------------------
    // It sets up the ring's barriers, meets the other warps once so that they see them, and starts
    // copying at once: W0 is the frozen base weight and does not depend on the work that precedes this
    // call on the stream, so only the other warps (which read x, the segments and the adapters) wait
    // for that work.  Lane r < 8 copies this stage's 4 KB of row r; a unit's chunks follow each other,
    // so the CTA walks its rows front to back, and the warp never waits for a round's epilogue, only
    // for free stages.
    if (producer) {
        if (lane == 0) {
            for (int s = 0; s < kS; ++s) {
                mbar_init(smem_u32(&ctrl->full[s]), 1);
                mbar_init(smem_u32(&ctrl->empty[s]), kDecConsumers);
            }
            mbar_init(smem_u32(&ctrl->ufull), kDecShrinkWarps * 32);
            mbar_init(smem_u32(&ctrl->bfull), 1);
            ctrl->abort = 0;
            ctrl->bad_offsets = 0;
            fence_mbar_init();
        }
        if (lane < 16) { ctrl->slot_of_row[lane] = -1; ctrl->b_of_row[lane] = -1; ctrl->b_lead[lane] = 0; ctrl->b_rows[lane] = 0; }
        asm volatile("bar.sync 4, %0;" ::"n"(kDecThreads) : "memory");   // the barriers are set up
        grid_launch_dependents();
        for (int round_begin = row_begin; round_begin < row_end && ok; round_begin += kDecRoundUnits * kDecUnitRows) {
            const int round_rows = min(kDecRoundUnits * kDecUnitRows, row_end - round_begin);
            const int nunits = (round_rows + kDecUnitRows - 1) / kDecUnitRows;
            const bool backwards = kMulti && (((round_begin - row_begin) / (kDecRoundUnits * kDecUnitRows)) & 1) != 0;
            for (int si = 0; si < nspans && ok; ++si) {
                const int sp = backwards ? nspans - 1 - si : si;   // (the consumers' order: see there)
                const int k_begin = sp * kSpan;
                const int span = min(kSpan, K - k_begin);
                const int nchunks = (span + kDecChunk - 1) / kDecChunk;
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
                        if (++stage == kS) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else {
        asm volatile("bar.sync 4, %0;" ::"n"(kDecThreads) : "memory");
        grid_dependency_wait();     // launched as a programmatic dependent: the work before this call is complete now
    }

    const int gq = lane >> 2, tq = lane & 3;
    bool u_ready = false;
    constexpr int kDecPerThread = kTwo ? 2 : 1;      // elements of y per consumer thread and round (16 x 32 or 8 x 32 over 256 threads)
    constexpr int kDecDefer = kDecDeferBytes / (kDecPerThread * kDecConsumers * 32 * 4);   // rounds whose expand can be put off
    static_assert(kDecRoundUnits * kDecUnitRows * (kTwo ? 16 : 8) <= kDecConsumers * 32 * kDecPerThread && kDecDefer >= 1, "elements per thread");
    int ndefer = 0;
    int span_loaded = -1;   // whose x fragments the registers hold

    // This warp's x fragments (chunk kc, k-steps warp*S .. warp*S+S-1 of a span) stay in registers.
    uint4 xa[kChunksPerSpan * kDecStepsPerChunk], xc[kTwo ? kChunksPerSpan * kDecStepsPerChunk : 1];
    // Fragment i of a chunk (i = 0..7 per warp) holds the 8 columns warp*256 + (i/2)*64 + tq*16 + (i&1)*8 ..: a lane's
    // fragments 2j and 2j+1 are 32 consecutive bytes of its row of x, so one 32-byte load fetches both and a warp's load
    // covers whole 128-byte lines (half as many requests to L2 as 16-byte loads).  The ring is read with the same
    // permutation, which a dot product does not see.
    const bool x_wide = ((reinterpret_cast<uintptr_t>(x) | (uintptr_t)((size_t)K * 2)) & 31u) == 0;
    auto load_x = [&](int k_begin, int span) {
        const bool ta = gq < T, tb = gq + 8 < T;
#pragma unroll
        for (int i = 0; i < kChunksPerSpan * kDecStepsPerChunk; i += 2) {
            const int c = (i / kDecStepsPerChunk) * kDecChunk + (warp * kDecStepsPerChunk + i % kDecStepsPerChunk) * 32 + tq * 16;
            const __nv_bfloat16* pa = x + (size_t)gq * K + k_begin + c;
            const __nv_bfloat16* pb = x + (size_t)(gq + 8) * K + k_begin + c;
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

    // ---- LoRA shrink, part of this kernel ---------------------------------------------------------------
    // Three extra warps do it while the other nine stream W0, so the base path never waits for it.
    // The first of them works out the slot of every row of x, raises the status flags and pulls the B
    // rows this CTA will need into L2.  Then the (token, j) dot products u = scale * x.A_j are dealt
    // out round-robin to the CTAs of the grid and, inside a CTA, to its three shrink warps: one warp per
    // dot product, sixteen 16-byte loads in flight per lane.  The results go to the exchange block in global
    // memory; a counter there tells every CTA when to look for them.  The consumers look at u only in their
    // first epilogue.
    unsigned int* sync_words = pj.sync_words;
    const bool shrinker = warp > kDecConsumers;
    // (The consumers do not hold their loads of x back until the lookup's few loads are on their way: that order was
    // worth 0.2 us once, and costs 0.1 - 0.4 us per call since the shrink warps no longer wait for a fence.)
    if (shrinker && G > 0) {
        const int sw = warp - kDecConsumers - 1;
        if (sw == 1) {
            // Which adapters this call names is known only after the lookup below, a memory round trip
            // from now, and their rows of A are cold.  When the table's live adapters are very few (their rows
            // of A together at most a 64th of W0), all of them are asked into L2 right now, ahead of the weight
            // stream, a row or two per CTA.  (With a 16th as the limit this was worth 0.3 us while the chain behind
            // the dot products was longer; now it changes nothing on a call that uses the adapters and costs
            // 0.1 - 0.2 us on one that does not, hence the narrow rule.  Taking the block out altogether was measured
            // too: the base-only call, which never runs it, came out 0.13 us slower, by code generation alone.)
            int rows_before = 0, my_rank[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int sl = lane + 32 * h;
                my_rank[h] = sl < snap.max_slots && sl < kMaxSlots ? (int)snap.rank[sl] : 0;
            }
            // running count of live rows in slot order: slots 0..31 first, then 32..63
            int incl0 = my_rank[0], incl1 = my_rank[1];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v0 = __shfl_up_sync(0xffffffffu, incl0, o), v1 = __shfl_up_sync(0xffffffffu, incl1, o);
                if (lane >= o) { incl0 += v0; incl1 += v1; }
            }
            const int total0 = __shfl_sync(0xffffffffu, incl0, 31);
            const int live_rows = total0 + __shfl_sync(0xffffffffu, incl1, 31);
            if ((long long)live_rows * K * 64 <= (long long)N * K) {
                // lane L of this CTA takes live row blockIdx + L * grid
                const int i = cta + lane * ncta;
                // find the slot holding live row i: the first whose inclusive count exceeds i
                const unsigned m0 = __ballot_sync(0xffffffffu, incl0 > 0);   // (dummy use keeps the shuffles converged)
                (void)m0;
                int slot = -1, j = 0;
                for (int src = 0; src < 32; ++src) {   // uniform loop: every lane reads every lane's counts
                    const int e0 = __shfl_sync(0xffffffffu, incl0, src), r0 = __shfl_sync(0xffffffffu, my_rank[0], src);
                    const int e1 = __shfl_sync(0xffffffffu, incl1, src) + total0, r1 = __shfl_sync(0xffffffffu, my_rank[1], src);
                    if (slot < 0 && i < e0 && i >= e0 - r0) { slot = src; j = i - (e0 - r0); }
                    if (slot < 0 && i < e1 && i >= e1 - r1) { slot = src + 32; j = i - (e1 - r1); }
                }
                if (i < live_rows && slot >= 0)
                    bulk_prefetch_l2(arenaA + ((size_t)slot * kRankPad + j) * K, (uint32_t)(K * 2));
                (void)rows_before;
            }
        }
        if (sw == kDecShrinkWarps - 1) {
            // this launch's mark: one more than that of the last launch that finished on these words
            unsigned last_epoch = 0;
            if (lane == 0) last_epoch = ld_relaxed_gpu(sync_words);
            for (int sl = lane; sl < kMaxSlots; sl += 32) lk->scale_s[sl] = snap.scale[sl];
            if (lane == 0) lk->epoch = last_epoch + 1u;
        }
        if (sw == 0) {
            // One memory round trip for everything the lookup needs: the segment arrays go to shared
            // memory (all loads issued before the first is used), the search then runs there.  Calls
            // with more segments than the cache holds search in global memory instead.  While the loads
            // are on their way, the slots' ranks and scales move from the kernel parameters to shared memory:
            // indexed reads of parameters are slow the first time, and everything later reads the copy.
            const bool by_token = token_slots != nullptr;   // one slot id per row of x instead of segments
            const bool cached = !by_token && G <= kDecSegCache;
            int my_row = lane;
            int so[kDecSegCache / 32 + 1], si[kDecSegCache / 32 + 1];
            if (cached) {
#pragma unroll
                for (int i = 0; i <= kDecSegCache / 32; ++i) {
                    const int g = lane + 32 * i;
                    so[i] = g <= G ? __ldg(seg_offsets + g) : 0;
                    si[i] = g < G ? __ldg(slot_ids + g) : -1;
                }
            }
            if (perm && lane < T) my_row = __ldg(perm + lane);
            int my_token_slot = -1;
            if (by_token && lane < T) {
                my_token_slot = __ldg(token_slots + lane);
                // the ids are adapter ids: the table's device map names the serving slot (-2: none, flagged below)
                if (adapter_map) my_token_slot = resolve_adapter(snap, adapter_map, my_token_slot);
            }
            for (int sl = lane; sl < kMaxSlots; sl += 32)   // ranks only: the scales (four more lines) come by another warp
                lk->rank_s[sl] = sl < snap.max_slots ? snap.rank[sl] : (uint8_t)0;
            if (lane == 0) lk->u_complete = 1;
            if (cached) {
#pragma unroll
                for (int i = 0; i <= kDecSegCache / 32; ++i) {
                    const int g = lane + 32 * i;
                    if (g <= G) lk->seg[g] = so[i];
                    if (g < G) lk->ids[g] = si[i];
                }
            }
            __syncwarp();
            auto rank_of = [&](int sl) { return (sl >= 0 && sl < kMaxSlots) ? (int)lk->rank_s[sl] : 0; };
            // (two separate code paths: written as one with selects, the compiler issues the global loads
            // of the uncached path unconditionally, a memory round trip on the critical path)
            int bad = 0, bad_slot = 0, bad_perm = 0, slot = -1;
            const int row = my_row;
            const bool row_ok = lane < T && row >= 0 && row < T;
            if (by_token) {   // same rule as the segmentation pass: an id that names no live adapter means none, and raises the flag
                if (lane < T) {
                    if (my_token_slot >= 0 && rank_of(my_token_slot) > 0) slot = my_token_slot;
                    else if (my_token_slot != -1) bad_slot = 1;
                }
            } else if (cached) {
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
                    const int s0 = __ldg(seg_offsets + g), s1 = __ldg(seg_offsets + g + 1), sl = __ldg(slot_ids + g);
                    if (s1 < s0 || s0 < 0 || s1 > T) bad = 1;
                    if (sl != -1 && s1 > s0 && rank_of(sl) == 0) bad_slot = 1;   // an empty segment may name anything
                }
                if (lane == 0 && (__ldg(seg_offsets) != 0 || __ldg(seg_offsets + G) != T)) bad = 1;
                if (row_ok) {
                    const int g = seg_upper(seg_offsets, G, lane);
                    if (g < G) { const int sl = __ldg(slot_ids + g); if (rank_of(sl) > 0) slot = sl; }
                }
            }
            bad = __any_sync(0xffffffffu, bad);
            bad_slot = __any_sync(0xffffffffu, bad_slot);
            if (!bad && lane < T) {
                if (row_ok) ctrl->slot_of_row[row] = slot; else bad_perm = 1;
            }
            bad_perm = __any_sync(0xffffffffu, bad_perm);
            if (lane == 0) {
                ctrl->bad_offsets = bad;
                const unsigned f = (bad ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_slot ? LML_FLAG_BAD_SLOT : 0u) |
                                   (bad_perm ? LML_FLAG_BAD_PERM : 0u);
                if (f && cta == 0) atomicOr(status, f);
            }
            __syncwarp();
            // Per row of x: rank, scale, and where its dot products end in the grid-wide numbering (rows
            // in order, j ascending inside a row, each row padded to a multiple of eight columns because
            // the expand reads u in groups of eight).
            {
                const int slot = lane < T ? ctrl->slot_of_row[lane] : -1;
                const int rank = slot >= 0 ? (int)lk->rank_s[slot] : 0;
                int end = (rank + 7) & ~7;
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, end, o);
                    if (lane >= o) end += v;
                }
                if (lane < 16) {
                    lk->dot_end[lane] = end;
                    lk->rank_of_row[lane] = rank;
                }
            }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");   // the slots are known
        // The dot products are dealt out in groups of one, two or four columns j of one row of x (a group
        // shares the row of x): group g belongs to CTA g mod grid.  A dot product's arithmetic is fixed, whoever
        // computes it: 96 "virtual threads" (the three shrink warps) each sum the 8-column chunks m, m + 96,
        // m + 192, ... of the row in order, each warp adds its threads' sums up with the butterfly, and the
        // result is (w0 + w1) + w2 times the scale.  The operands of a whole group (up to six 16-byte chunks of x
        // and of each row of A per thread and step: 4608 columns) are in flight at once, in registers, so a group costs
        // one memory round trip per step.  (Groups staged in shared memory by asynchronous copies were measured slower:
        // 1.1 us per call for pairs at 12 and 16 tokens, 0.6 - 2.3 us for groups of four.)  A result is published as one
        // 64-bit store (value and this launch's mark) and a relaxed add on the grid-wide counter: nobody waits for a fence.
        const int total = lk->dot_end[15];
        // Group size: the smallest of 1, 2, 4 that gives every CTA at most one group (a group costs a memory
        // round trip, but also (1 + size) x 8 KB through the load path of its CTA), else 4.
        const int gsize = total <= ncta ? 1 : (total <= 2 * ncta ? 2 : kDecDotGroup);
        const int ngroups = total / gsize;
        const int me = tid - (kDecConsumers + 1) * 32;   // 0 .. 95
        // Where the expand will find its B operand: worked out by the first shrink warp in the shadow of its first dot
        // product's loads (0.6 us of single-warp work that nothing ahead of the epilogue waits for; CTAs without a dot
        // product of their own do it after the others').
        bool booked = false;
        auto book_once = [&]() {   // (called by whole warps only: the first shrink warp shuffles in here)
            if (sw == 0 && !booked) {
                __syncwarp();
                const int slot = lane < T ? ctrl->slot_of_row[lane] : -1;
                const int rank = slot >= 0 ? (int)lk->rank_s[slot] : 0;
                // The expand reads, per distinct slot, the first ceil(rank / 8) 16-byte chunks of this CTA's
                // rows of B.  Those go into the staging buffer, one block per distinct slot as long as they fit; the
                // first row of x with a slot stands for the slot's block.  A slot of rank <= 16 comes in right here as
                // one bulk copy of this CTA's rows of the compact arena (32 bytes each, row after row): a single
                // instruction of this warp for all slots, where the chunk-by-chunk copies further down cost the shrink
                // warps about 0.2 us per slot.  The other blocks are chunk-major ([chunk][row]:
                // consecutive threads of the epilogue read consecutive 16 bytes) and are filled by stage_b.
                const unsigned same = __match_any_sync(0xffffffffu, slot);
                const int first = __ffs(same) - 1;
                const bool leader = rank > 0 && first == lane;
                const int rows_cta = row_end - row_begin;
                const bool whole_rows = rank <= kRankCompact;
                const int chunks = leader ? rows_cta * (whole_rows ? kRankCompact / 8 : ((rank + 7) >> 3)) : 0;
                int base = chunks;
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, base, o);
                    if (lane >= o) base += v;
                }
                const int fits = base * 16 <= kDotBytes;   // (inclusive end of this block)
                const int my_off = __shfl_sync(0xffffffffu, fits ? (base - chunks) * 16 : -1, first);
                if (lane < 16) {
                    ctrl->b_of_row[lane] = rank > 0 ? my_off : -1;
                    ctrl->b_lead[lane] = leader ? 1 : 0;
                    ctrl->b_rows[lane] = rank > 0 && whole_rows && my_off >= 0 ? 1 : 0;
                    lk->row_info[lane] = rank > 0 ? (0x80000000u | (unsigned)slot | ((unsigned)((rank + 7) >> 3) << 8) | (whole_rows ? 1u << 12 : 0u) |
                                                     (my_off >= 0 ? (1u << 13) | ((unsigned)(my_off >> 4) << 16) : 0u))
                                                  : 0u;
                }
                const bool bulk = leader && whole_rows && fits && lane < 16;
                int bulk_bytes = bulk ? chunks * 16 : 0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) bulk_bytes += __shfl_xor_sync(0xffffffffu, bulk_bytes, o);
                if (lane == 0) mbar_arrive_expect_tx(smem_u32(&ctrl->bfull), (uint32_t)bulk_bytes);
                __syncwarp();
                if (bulk)
                    bulk_copy_g2s(smem_u32(dot_s) + (uint32_t)((base - chunks) * 16), arenaBc + ((size_t)slot * N + row_begin) * kRankCompact,
                                  (uint32_t)(chunks * 16), smem_u32(&ctrl->bfull));
            }
            booked = true;
        };
        // Brings the blocks of B into the staging buffer (16-byte asynchronous copies, all in flight at
        // once); blocks that did not fit are asked into L2 and read from there by the epilogue.
        auto stage_b = [&]() {
            const int rows_cta = row_end - row_begin;
            for (int t = 0; t < T; ++t) {
                if (!ctrl->b_lead[t] || ctrl->b_rows[t]) continue;   // (whole rows came by bulk copy)
                const int r8 = (lk->rank_of_row[t] + 7) >> 3;
                // (ranks up to 16 are read from the compact copy of B: 32-byte rows back to back, not a quarter of a padded row each)
                const bool compact = lk->rank_of_row[t] <= kRankCompact;
                const int pitch = compact ? kRankCompact * 2 : kRankPad * 2;
                const char* b = compact ? reinterpret_cast<const char*>(arenaBc + ((size_t)ctrl->slot_of_row[t] * N + row_begin) * kRankCompact)
                                        : reinterpret_cast<const char*>(arenaB + ((size_t)ctrl->slot_of_row[t] * N + row_begin) * kRankPad);
                const int off = ctrl->b_of_row[t];
                if (off >= 0) {
                    for (int i = me; i < rows_cta * r8; i += kDecShrinkWarps * 32) {
                        const int c = i / rows_cta, r = i - c * rows_cta;
                        cp_async_16(smem_u32(dot_s) + off + i * 16, b + (size_t)r * pitch + c * 16);
                    }
                } else {
                    for (int r = me; r < rows_cta; r += kDecShrinkWarps * 32) prefetch_l2(b + (size_t)r * pitch);
                }
            }
        };
        // A single dot product per CTA (few tokens, rank 16: the usual decode call).
        auto single = [&](int d, int& t, int& j) {
            t = 0;
            while (lk->dot_end[t] <= d) ++t;
            j = d - (t > 0 ? lk->dot_end[t - 1] : 0);
            const bool real = j < lk->rank_of_row[t];
            if (real) {
                const __nv_bfloat16* xr = x + (size_t)t * K;
                const __nv_bfloat16* ar = arenaA + ((size_t)ctrl->slot_of_row[t] * kRankPad + j) * K;
                constexpr int kPer = 6, kStride = kDecShrinkWarps * 32 * 8;
                float dot = 0.f;
                for (int kb = me * 8, step = 0; step == 0 || kb < K; kb += kPer * kStride, ++step) {   // (every thread takes the first step: see book_once)
                    uint4 xv[kPer], av[kPer];
#pragma unroll
                    for (int i = 0; i < kPer; ++i) {
                        const int k0 = kb + i * kStride;
                        const bool ok_k = k0 < K;
                        xv[i] = ok_k ? ldg_nc_v4(xr + k0) : make_uint4(0, 0, 0, 0);
                        av[i] = ok_k ? ldg_nc_v4(ar + k0) : make_uint4(0, 0, 0, 0);
                    }
                    book_once();   // (while the loads are on their way)
#pragma unroll
                    for (int i = 0; i < kPer; ++i) {
                        if (kb + i * kStride < K) {
                            float p = 0.f;
                            p = fmaf(bf16_lo(xv[i].x), bf16_lo(av[i].x), p); p = fmaf(bf16_hi(xv[i].x), bf16_hi(av[i].x), p);
                            p = fmaf(bf16_lo(xv[i].y), bf16_lo(av[i].y), p); p = fmaf(bf16_hi(xv[i].y), bf16_hi(av[i].y), p);
                            p = fmaf(bf16_lo(xv[i].z), bf16_lo(av[i].z), p); p = fmaf(bf16_hi(xv[i].z), bf16_hi(av[i].z), p);
                            p = fmaf(bf16_lo(xv[i].w), bf16_lo(av[i].w), p); p = fmaf(bf16_hi(xv[i].w), bf16_hi(av[i].w), p);
                            dot += p;
                        }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                if (lane == 0) lk->dot_part[0][sw] = dot;
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");
            const float val = real ? ((lk->dot_part[0][0] + lk->dot_part[0][1]) + lk->dot_part[0][2]) * lk->scale_s[ctrl->slot_of_row[t]] : 0.f;
            asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");   // dot_part is free again
            return val;
        };
        // A group of two or four dot products of one row of x, operands in registers like the single one: each virtual
        // thread sums the same chunks in the same order, so a dot product has the same bits whichever path computes it.
        auto regs_group = [&](auto ng_tag, int g, float (&val)[kDecDotGroup], int& t, int& j0) {
            constexpr int NG = decltype(ng_tag)::value;
            const int d0 = g * NG;
            t = 0;
            while (lk->dot_end[t] <= d0) ++t;
            j0 = d0 - (t > 0 ? lk->dot_end[t - 1] : 0);
            const int nreal = max(0, min(NG, lk->rank_of_row[t] - j0));
            float dot[NG];
#pragma unroll
            for (int d = 0; d < NG; ++d) dot[d] = 0.f;
            if (nreal > 0) {
                const __nv_bfloat16* xr = x + (size_t)t * K;
                const __nv_bfloat16* ar = arenaA + ((size_t)ctrl->slot_of_row[t] * kRankPad + j0) * K;
                constexpr int kPer = 6, kStride = kDecShrinkWarps * 32 * 8;
                for (int kb = me * 8, step = 0; step == 0 || kb < K; kb += kPer * kStride, ++step) {   // (every thread takes the first step: see book_once)
                    uint4 xv[kPer], av[NG][kPer];
#pragma unroll
                    for (int i = 0; i < kPer; ++i) {
                        const int k0 = kb + i * kStride;
                        const bool ok_k = k0 < K;
                        xv[i] = ok_k ? ldg_nc_v4(xr + k0) : make_uint4(0, 0, 0, 0);
#pragma unroll
                        for (int d = 0; d < NG; ++d)
                            av[d][i] = ok_k && d < nreal ? ldg_nc_v4(ar + (size_t)d * K + k0) : make_uint4(0, 0, 0, 0);
                    }
                    book_once();   // (while the loads are on their way)
#pragma unroll
                    for (int i = 0; i < kPer; ++i) {
                        if (kb + i * kStride < K) {
#pragma unroll
                            for (int d = 0; d < NG; ++d) {
                                float p = 0.f;
                                p = fmaf(bf16_lo(xv[i].x), bf16_lo(av[d][i].x), p); p = fmaf(bf16_hi(xv[i].x), bf16_hi(av[d][i].x), p);
                                p = fmaf(bf16_lo(xv[i].y), bf16_lo(av[d][i].y), p); p = fmaf(bf16_hi(xv[i].y), bf16_hi(av[d][i].y), p);
                                p = fmaf(bf16_lo(xv[i].z), bf16_lo(av[d][i].z), p); p = fmaf(bf16_hi(xv[i].z), bf16_hi(av[d][i].z), p);
                                p = fmaf(bf16_lo(xv[i].w), bf16_lo(av[d][i].w), p); p = fmaf(bf16_hi(xv[i].w), bf16_hi(av[d][i].w), p);
                                dot[d] += p;
                            }
                        }
                    }
                }
#pragma unroll
                for (int d = 0; d < NG; ++d) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) dot[d] += __shfl_xor_sync(0xffffffffu, dot[d], o);
                    if (lane == 0) lk->dot_part[d][sw] = dot[d];
                }
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");
#pragma unroll
            for (int i = 0; i < kDecDotGroup; ++i)
                val[i] = i < nreal ? ((lk->dot_part[i][0] + lk->dot_part[i][1]) + lk->dot_part[i][2]) * lk->scale_s[ctrl->slot_of_row[t]] : 0.f;
            asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");   // dot_part is free again
        };
        auto group = [&](int g, float (&val)[kDecDotGroup], int& t, int& j0) {
            if (gsize == 4) regs_group(std::integral_constant<int, 4>{}, g, val, t, j0);
            else regs_group(std::integral_constant<int, 2>{}, g, val, t, j0);
        };
        const long long t_shrink = clock64();
        const unsigned epoch = lk->epoch;
        if (gsize == 1) {
            if (cta < total) {
                int t, j;
                const float val = single(cta, t, j);
                if (me == 0) {
                    st_relaxed_gpu_b64(u + t * kRankPad + j, pack_u(val, epoch));
                    red_relaxed_gpu_add(sync_words + 2, 1u);
                }
            }
        } else
        for (int g = cta; g < ngroups; g += ncta) {
            float val[kDecDotGroup];
            int t, j0;
            group(g, val, t, j0);
            if (me == 0) {
                for (int i = 0; i < gsize; ++i) st_relaxed_gpu_b64(u + t * kRankPad + j0 + i, pack_u(val[i], epoch));
                red_relaxed_gpu_add(sync_words + 2, (unsigned)gsize);
            }
        }
        book_once();   // (a CTA without a dot product of its own, or whose group had only padding columns)
        asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");   // the blocks of B are placed
        stage_b();     // the chunk-by-chunk copies (ranks above 16); the staging buffer is theirs alone
        // Collect all of u in shared memory for the consumers' epilogue, off their critical path.  The
        // other CTAs' shares normally arrive within microseconds and are then read from global memory.
        // But this CTA never depends on them: nothing guarantees that the whole grid is resident at once
        // (the launch is an ordinary one, so that it can start while its predecessor drains), so after a
        // bounded wait it simply computes every dot product itself, with the same arithmetic and hence the
        // same bits, finishes and makes room for whichever CTAs have not started yet.
        // (The wait ends when HALF of the entries are counted: the read of the entries that follows takes a round trip of
        // its own, by the end of which the rest has usually arrived, and what has not is asked for again.  Worth 0.1 -
        // 0.2 us per call against waiting for all of them; a quarter or an eighth is no better.)
        if (sw == 0 && lane == 0) {
            while (ld_relaxed_gpu(sync_words + 2) < (unsigned)((total + 1) / 2)) {
                if (clock64() - t_shrink > (long long)patience) { lk->u_complete = 0; break; }
            }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");
        if (lk->u_complete) {
            // Every entry of u is a 64-bit word, the value beside the mark of the launch that wrote it, and is written and
            // read as one: an entry that carries this launch's mark is this launch's value, whatever order the stores and
            // the counter's adds became visible in (the counter only says when looking is worth it: 148 CTAs that poll the
            // entries themselves from the start were measured 0.5 us and more slower than the counter they replaced).  A thread takes pairs
            // of entries (16 bytes) of the columns that the expand reads, has all its loads in flight at once and asks
            // again for what was not there yet.
            constexpr int kPairs = (16 * kRankPad / 2 + kDecShrinkWarps * 32 - 1) / (kDecShrinkWarps * 32);   // 6
            unsigned pending = 0;
#pragma unroll
            for (int k = 0; k < kPairs; ++k) {
                const int i = me + k * kDecShrinkWarps * 32;
                const int t = i / (kRankPad / 2), j = (i % (kRankPad / 2)) * 2;
                if (t < T && j < ((lk->rank_of_row[t & 15] + 7) & ~7)) pending |= 1u << k;
            }
            while (pending) {
                unsigned long long e0[kPairs], e1[kPairs];
#pragma unroll
                for (int k = 0; k < kPairs; ++k)
                    if (pending >> k & 1u) ld_relaxed_gpu_v2_b64(u + 2 * (me + k * kDecShrinkWarps * 32), e0[k], e1[k]);
#pragma unroll
                for (int k = 0; k < kPairs; ++k) {
                    if ((pending >> k & 1u) && (unsigned)(e0[k] >> 32) == epoch && (unsigned)(e1[k] >> 32) == epoch) {
                        reinterpret_cast<float2*>(u_s)[me + k * kDecShrinkWarps * 32] =
                            make_float2(__uint_as_float((unsigned)e0[k]), __uint_as_float((unsigned)e1[k]));
                        pending &= ~(1u << k);
                    }
                }
                if (pending && clock64() - t_shrink > (long long)patience) { lk->u_complete = 0; break; }
            }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kDecShrinkWarps * 32) : "memory");
        if (lk->u_complete) {
            // (u_s holds every column that the expand reads)
        } else if (gsize == 1) {
            for (int d = 0; d < total; ++d) {
                int t, j;
                const float val = single(d, t, j);
                if (me == 0) u_s[t * kRankPad + j] = val;
            }
        } else {
            for (int g = 0; g < ngroups; ++g) {
                float val[kDecDotGroup];
                int t, j0;
                group(g, val, t, j0);
                if (me == 0) for (int i = 0; i < gsize; ++i) u_s[t * kRankPad + j0 + i] = val[i];
            }
        }
        cp_async_wait_all();   // this thread's chunks of B have landed
        mbar_wait_warp(smem_u32(&ctrl->bfull), 0u, abort);   // and so have the bulk copies (on a give-up the flag is up: the call reports it)
        // tell the consumers that u_s, slot_of_row, bad_offsets and the copies of B are final (each thread
        // releases what it wrote)
        if (kPutOff) mbar_arrive(smem_u32(&ctrl->ufull));   // (the consumers can test this one without waiting)
        else asm volatile("bar.arrive 3, %0;" ::"n"((kDecConsumers + kDecShrinkWarps) * 32) : "memory");
        // Every CTA signs off once it has its copy of u and has published its own share; the last one makes this
        // launch's mark the table's last one, so that the next call on this table takes the next mark, and puts the
        // counter back to zero.
        if (sw == 0 && lane == 0) {
            // (no fence: this thread's own polls are complete, and what the other threads still read stays as it is
            // until the next launch, which begins after this grid has finished)
            if (atomicAdd(sync_words + 1, 1u) == (unsigned)ncta - 1u) {
                if (epoch == 0xffffffffu) {   // the marks start over: no entry may keep one of the last round (a thread that still
                                              // reads then misses its entries, and its CTA computes u itself: same bits)
                    for (int i = 0; i < kDecExchEntries; ++i) u[i] = 0ull;
                    __threadfence();
                    sync_words[0] = 0u;
                } else {
                    sync_words[0] = epoch;
                }
                sync_words[1] = 0u;
                sync_words[2] = 0u;
            }
        }
    }

    for (int round_begin = consumer ? row_begin : row_end; round_begin < row_end; round_begin += kDecRoundUnits * kDecUnitRows) {
        const int round_rows = min(kDecRoundUnits * kDecUnitRows, row_end - round_begin);
        const int nunits = (round_rows + kDecUnitRows - 1) / kDecUnitRows;
        // The spans are walked forwards in even rounds and backwards in odd ones: the x fragments of the
        // span a round ends with are the ones the next round starts with and need no reload (with a
        // single span, x is loaded once per CTA).
        const bool backwards = kMulti && (((round_begin - row_begin) / (kDecRoundUnits * kDecUnitRows)) & 1) != 0;
        for (int si = 0; si < nspans; ++si) {
            const int sp = backwards ? nspans - 1 - si : si;
            const int k_begin = sp * kSpan;
            const int span = min(kSpan, K - k_begin);
            const int nchunks = (span + kDecChunk - 1) / kDecChunk;
            {
                // ---------------------------------------------------------- consumer warps
                // this warp's k-steps of the span: chunk kc, steps warp*4 .. warp*4+3.  The x fragments
                // live in registers for every row of the round.
                if (!kMulti) load_x(k_begin, span);
                else if (sp != span_loaded) { load_x(k_begin, span); span_loaded = sp; }
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
                                const uint32_t wbase = ring + stage * kDecStageBytes + gq * kDecRowPitch + tq * 32 + warp * (kDecStepsPerChunk * 64);
                                // all of the stage's operand reads first, then the stage can go back to the producer
                                // before the MMAs run
                                uint4 w[kDecStepsPerChunk];
                                if (rows == kDecUnitRows && span - kc * kDecChunk >= kDecChunk) {
                                    // a full stage (all but the ragged edges): no predicates
#pragma unroll
                                    for (int i = 0; i < kDecStepsPerChunk; ++i)
                                        w[i] = lds128(wbase + (uint32_t)((i >> 1) * 128 + (i & 1) * 16));
#pragma unroll
                                    for (int i = 0; i < kDecStepsPerChunk; ++i) {
                                        const uint4 a0 = xa[kc * kDecStepsPerChunk + i];
                                        const uint4 a1 = kTwo ? xc[kc * kDecStepsPerChunk + i] : make_uint4(0, 0, 0, 0);
                                        mma_bf16_16816(acc4[(2 * i) & 3], a0.x, a1.x, a0.y, a1.y, w[i].x, w[i].y);
                                        mma_bf16_16816(acc4[(2 * i + 1) & 3], a0.z, a1.z, a0.w, a1.w, w[i].z, w[i].w);
                                    }
                                } else {
#pragma unroll
                                    for (int i = 0; i < kDecStepsPerChunk; ++i) {
                                        const int c0 = kc * kDecChunk + (warp * kDecStepsPerChunk + (i & ~1)) * 32;   // the pair's 64 columns start here
                                        w[i] = (rv && c0 + tq * 16 + (i & 1) * 8 < span) ? lds128(wbase + (uint32_t)((i >> 1) * 128 + (i & 1) * 16))
                                                                                         : make_uint4(0, 0, 0, 0);
                                    }
#pragma unroll
                                    for (int i = 0; i < kDecStepsPerChunk; ++i) {
                                        const int c0 = kc * kDecChunk + (warp * kDecStepsPerChunk + (i & ~1)) * 32;
                                        if (c0 < span) {   // uniform across the warp: all lanes issue the MMAs or none
                                            const uint4 a0 = xa[kc * kDecStepsPerChunk + i];
                                            const uint4 a1 = kTwo ? xc[kc * kDecStepsPerChunk + i] : make_uint4(0, 0, 0, 0);
                                            mma_bf16_16816(acc4[(2 * i) & 3], a0.x, a1.x, a0.y, a1.y, w[i].x, w[i].y);
                                            mma_bf16_16816(acc4[(2 * i + 1) & 3], a0.z, a1.z, a0.w, a1.w, w[i].z, w[i].w);
                                        }
                                    }
                                }
                                __syncwarp();
                                if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[stage]));
                                if (++stage == kS) { stage = 0; phase ^= 1u; }
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
                    if (si == 0) {
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
        // The expand needs u, which the whole grid computes: it is there a few microseconds after the call
        // before this one has ended everywhere.  A CTA with several rounds does not wait for it: until u
        // has arrived, each thread keeps the base sums of its elements of up to kDecDefer rounds in
        // shared memory (the same thread finishes them later), and only then, or in its last round, it waits.
        // This thread's elements of the round (token t, row j of the round) and their base sums, before any wait for u.
        float base_v[kDecPerThread];
        int el_t[kDecPerThread], el_j[kDecPerThread];
        if (consumer && ok) {
            const int per_token = nunits * kDecUnitRows;
#pragma unroll
            for (int i = 0; i < kDecPerThread; ++i) {
                const int e = tid + i * kDecConsumers * 32;   // consecutive threads: consecutive rows
                base_v[i] = 0.f;
                el_t[i] = -1;
                el_j[i] = 0;
                if (e < T * per_token) {
                    const int t = e / per_token, j = e % per_token;
                    const int un = j / kDecUnitRows, r = j % kDecUnitRows;
                    float v = 0.f;
#pragma unroll
                    for (int w = 0; w < kDecConsumers; ++w) v += slots[(un * kDecConsumers + w) * kDecSlotFloats + t * 8 + r];
                    base_v[i] = v;
                    el_t[i] = t;
                    el_j[i] = j;
                }
            }
        }
        if (!kPutOff) {
            if (consumer && G > 0 && !u_ready) {   // first epilogue: the shrink warps have staged u in shared memory
                asm volatile("bar.sync 3, %0;" ::"n"((kDecConsumers + kDecShrinkWarps) * 32) : "memory");
                u_ready = true;
            }
        } else if (consumer && ok && G > 0 && !u_ready) {
            const bool last_round = round_begin + kDecRoundUnits * kDecUnitRows >= row_end;
            if (last_round || ndefer == kDecDefer) {
                int there = 1;   // (polling: the flip is seen within a few cycles, no wake-up)
                if (lane == 0) there = mbar_wait_spin(smem_u32(&ctrl->ufull), 0u, abort) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, there, 0) != 0;
                u_ready = ok;
            } else {
                int there = lane == 0 ? (mbar_test_wait(smem_u32(&ctrl->ufull), 0u) ? 1 : 0) : 0;
                u_ready = __shfl_sync(0xffffffffu, there, 0) != 0;
            }
        }
        if (consumer && ok) {
            const bool lora = G > 0 && u_ready && ctrl->bad_offsets == 0;
            const int rows_cta = row_end - row_begin;
            // y[t][n] = base sum + u_t . B_slot[n] (the first ceil(rank / 8) chunks of the row), rounded once
            auto finish = [&](int t, int n, float v) {
                const unsigned info = lora ? lk->row_info[t] : 0u;
                if (info >> 31) {
                    const int slot = (int)(info & 0xffu), r8 = (int)((info >> 8) & 0xfu);
                    const bool compact = (info >> 12 & 1u) != 0, staged = (info >> 13 & 1u) != 0;
                    const float4* up = reinterpret_cast<const float4*>(u_s + t * kRankPad);
                    float d = 0.f;
                    auto fma8 = [&](const uint4& b, const float4& u0, const float4& u1) {
                        d = fmaf(u0.x, bf16_lo(b.x), d); d = fmaf(u0.y, bf16_hi(b.x), d);
                        d = fmaf(u0.z, bf16_lo(b.y), d); d = fmaf(u0.w, bf16_hi(b.y), d);
                        d = fmaf(u1.x, bf16_lo(b.z), d); d = fmaf(u1.y, bf16_hi(b.z), d);
                        d = fmaf(u1.z, bf16_lo(b.w), d); d = fmaf(u1.w, bf16_hi(b.w), d);
                    };
                    const uint4* bs = reinterpret_cast<const uint4*>(dot_s + ((info >> 16) & 0xfffu) * 16u);
                    if (staged && compact) {
                        // the usual case (whole 32-byte rows by bulk copy): everything is asked for at once, then summed in order
                        const uint4* br = bs + (n - row_begin) * (kRankCompact / 8);
                        const bool two = r8 > 1;
                        const uint4 b0 = br[0];
                        const uint4 b1 = two ? br[1] : make_uint4(0, 0, 0, 0);
                        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                        const float4 u0 = up[0], u1 = up[1], u2 = two ? up[2] : z, u3 = two ? up[3] : z;
                        fma8(b0, u0, u1);
                        if (two) fma8(b1, u2, u3);
                    } else if (staged) {   // (two loops: with a select inside one loop the global loads no longer overlap)
                        for (int c = 0; c < r8; ++c) fma8(bs[c * rows_cta + (n - row_begin)], up[2 * c], up[2 * c + 1]);
                    } else {
                        const uint4* bp = compact ? reinterpret_cast<const uint4*>(arenaBc + ((size_t)slot * N + n) * kRankCompact)
                                                  : reinterpret_cast<const uint4*>(arenaB + ((size_t)slot * N + n) * kRankPad);
                        for (int c = 0; c < r8; ++c) fma8(ldg_nc_v4(bp + c), up[2 * c], up[2 * c + 1]);
                    }
                    v += d;
                }
                y[(size_t)t * N + n] = __float2bfloat16_rn(v);
            };
            if (kPutOff && G > 0 && !u_ready) {   // put this round off (a full round: the last one waits)
#pragma unroll
                for (int i = 0; i < kDecPerThread; ++i)
                    if (el_t[i] >= 0) defer_s[ndefer * (kDecPerThread * kDecConsumers * 32) + tid + i * kDecConsumers * 32] = base_v[i];   // read back by this very thread
                ++ndefer;
            } else {
                if (kPutOff && ndefer > 0) {   // the rounds that were put off
                    constexpr int kFull = kDecRoundUnits * kDecUnitRows;
                    for (int dd = 0; dd < ndefer; ++dd)
                        for (int e = tid; e < T * kFull; e += kDecConsumers * 32)
                            finish(e / kFull, round_begin - (ndefer - dd) * kFull + e % kFull,
                                   defer_s[dd * (kDecPerThread * kDecConsumers * 32) + e]);
                    ndefer = 0;
                }
#pragma unroll
                for (int i = 0; i < kDecPerThread; ++i)
                    if (el_t[i] >= 0 && el_j[i] < round_rows) finish(el_t[i], round_begin + el_j[i], base_v[i]);
            }
        }
        if (consumer) asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers * 32) : "memory");   // slots are free for the next round
    }
    if (ctrl->abort) __nanosleep(50000);   // gave up: let copies still in flight land before the CTA goes away
    if (tid == 0 && ctrl->abort) atomicOr(status, LML_FLAG_TIMEOUT);
}

namespace {
// How long (SM clock cycles) a CTA waits for the other CTAs' share of u before it computes all of it
// itself: far longer than the normal hand-over takes (a few microseconds), short enough that a grid
// that cannot be resident all at once still finishes promptly.  LML_DECODE_PATIENCE overrides it (the
// tests set 0 to run the self-sufficient path on purpose).
int g_dec_patience = 100000;
}  // namespace

cudaError_t decode_init()
{
    if (const char* e = getenv("LML_DECODE_PATIENCE")) g_dec_patience = atoi(e) < 0 ? 0 : atoi(e);
    cudaError_t e = cudaSuccess;
    auto set = [&](auto kernel) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecSmemBytes);
    };
    set(decode_main_kernel<false, false, false, 1>); set(decode_main_kernel<false, true, false, 1>); set(decode_main_kernel<false, true, true, 1>);
    set(decode_main_kernel<true, false, false, 1>);  set(decode_main_kernel<true, true, false, 1>);  set(decode_main_kernel<true, true, true, 1>);
    set(decode_main_kernel<false, false, false, kDecMaxProj>); set(decode_main_kernel<false, true, false, kDecMaxProj>); set(decode_main_kernel<false, true, true, kDecMaxProj>);
    set(decode_main_kernel<true, false, false, kDecMaxProj>);  set(decode_main_kernel<true, true, false, kDecMaxProj>);  set(decode_main_kernel<true, true, true, kDecMaxProj>);
    auto set_base = [&](auto kernel) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfg<kDecVarBase>::kSmemBytes);
    };
    set_base(decode_main_kernel<false, false, false, 1, kDecVarBase>); set_base(decode_main_kernel<false, true, false, 1, kDecVarBase>);
    set_base(decode_main_kernel<true, false, false, 1, kDecVarBase>);  set_base(decode_main_kernel<true, true, false, 1, kDecVarBase>);
    auto set_small = [&](auto kernel) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfg<kDecVarSmall>::kSmemBytes);
    };
    set_small(decode_main_kernel<false, false, false, 1, kDecVarSmall>); set_small(decode_main_kernel<false, true, true, 1, kDecVarSmall>);
    set_small(decode_main_kernel<true, false, false, 1, kDecVarSmall>);  set_small(decode_main_kernel<true, true, true, 1, kDecVarSmall>);
    return e;
}

int decode_patience() { return g_dec_patience; }

namespace {

void fill_proj(DecProj& pj, const Arena& ar, const DecodeArgs& a)
{
    pj.arenaA = ar.A; pj.arenaB = ar.B; pj.arenaBc = ar.Bc;
    pj.W0 = (const __nv_bfloat16*)a.W0;
    pj.x = (const __nv_bfloat16*)a.x;
    pj.T = a.T;
    pj.snap_idx = 0;
    pj.y = (__nv_bfloat16*)a.y;
    pj.u = a.exch ? a.exch : ar.dec_u;
    pj.seg_offsets = a.seg_offsets; pj.slot_ids = a.slot_ids; pj.perm = a.perm; pj.token_slots = a.token_slots;
    pj.adapter_map = a.by_adapter ? ar.adapter_map : nullptr;
    pj.status = ar.status;
    pj.sync_words = reinterpret_cast<unsigned int*>(pj.u + kDecExchEntries);
    pj.N = a.d_out; pj.G = a.G;
}

// An ordinary launch, as a programmatic dependent of whatever precedes it on the stream (the kernel waits for that
// work itself, after it has started on W0).  The CTAs hand one another their share of u, but none of them depends on
// the others being resident (see the kernel), so no cooperative launch is needed, and the kernel can start while its
// predecessor drains.  Three builds of the kernel per token count: CTAs with one round of rows (the plain loop), with
// several rounds (x is kept between rounds), and with several rounds and adapters (the expand of early rounds is put
// off until u has arrived).
template <int kP>
cudaError_t launch_decode_grid(const DecLaunch<kP>& prm, int grid, int rows_per_cta, bool adapters, int max_T, cudaStream_t stream,
                               bool small_blocks = false)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kDecThreads);
    cfg.dynamicSmemBytes = kDecSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool multi = rows_per_cta > kDecRoundUnits * kDecUnitRows;
    const bool put_off = multi && adapters;
    auto launch = [&](auto kernel) { return cudaLaunchKernelEx(&cfg, kernel, prm); };
    if constexpr (kP == 1) {
        if (!adapters) {   // no adapter anywhere in the call: the build with the deeper ring and no staging buffer
            cfg.dynamicSmemBytes = DecCfg<kDecVarBase>::kSmemBytes;
            if (max_T > 8) return multi ? launch(decode_main_kernel<true, true, false, 1, kDecVarBase>) : launch(decode_main_kernel<true, false, false, 1, kDecVarBase>);
            return multi ? launch(decode_main_kernel<false, true, false, 1, kDecVarBase>) : launch(decode_main_kernel<false, false, false, 1, kDecVarBase>);
        }
        if (small_blocks) {   // the blocks of B are sure to fit in the small staging buffer: the build with the deeper ring
            cfg.dynamicSmemBytes = DecCfg<kDecVarSmall>::kSmemBytes;
            if (max_T > 8) return multi ? launch(decode_main_kernel<true, true, true, 1, kDecVarSmall>) : launch(decode_main_kernel<true, false, false, 1, kDecVarSmall>);
            return multi ? launch(decode_main_kernel<false, true, true, 1, kDecVarSmall>) : launch(decode_main_kernel<false, false, false, 1, kDecVarSmall>);
        }
    }
    if (max_T > 8)
        return put_off ? launch(decode_main_kernel<true, true, true, kP>)
                       : (multi ? launch(decode_main_kernel<true, true, false, kP>) : launch(decode_main_kernel<true, false, false, kP>));
    return put_off ? launch(decode_main_kernel<false, true, true, kP>)
                   : (multi ? launch(decode_main_kernel<false, true, false, kP>) : launch(decode_main_kernel<false, false, false, kP>));
}

}  // namespace

cudaError_t launch_decode(const Arena& ar, const SlotSnapshot& snap, const DecodeArgs& a, cudaStream_t stream,
                          int* launches)
{
    *launches = 0;
    const int row_pairs = (a.d_out + 1) / 2;   // at least two rows per CTA
    const int grid = row_pairs < a.num_sms ? row_pairs : a.num_sms;
    DecLaunch<1> prm;
    prm.snap[0] = snap;
    fill_proj(prm.proj[0], ar, a);
    prm.proj[0].cta_begin = 0; prm.proj[0].cta_count = grid;
    prm.x = (const __nv_bfloat16*)a.x;
    prm.T = a.T; prm.K = a.d_in; prm.P = 1; prm.patience = g_dec_patience;
    // Worst case of what the expand's copies of B take per CTA: a block per distinct slot (at most one per token, and no
    // more than the table has live), the widest block that any live slot can have.
    const int rows_per_cta = (a.d_out + grid - 1) / grid;
    int live = 0, widest = 0;
    for (int sl = 0; sl < snap.max_slots && sl < kMaxSlots; ++sl) {
        const int r = snap.rank[sl];
        if (r == 0) continue;
        ++live;
        const int per_row = r <= kRankCompact ? kRankCompact * 2 : ((r + 7) >> 3) * 16;
        widest = per_row > widest ? per_row : widest;
    }
    const int blocks = a.T < live ? a.T : live;
    const bool small_blocks = a.G > 0 && (long long)blocks * rows_per_cta * widest <= kDecDotBytesSmall;
    const cudaError_t e = launch_decode_grid<1>(prm, grid, rows_per_cta, a.G > 0, a.T, stream, small_blocks);
    if (e == cudaSuccess) ++*launches;
    return e;
}

// Several projections of one decode step (the same x, T and d_in) in one launch: the SMs are dealt out in proportion to
// the projections' rows (every projection gets at least one CTA, none more than it has pairs of rows).
cudaError_t launch_decode_multi(const Arena* const* ars, const SlotSnapshot* snaps, const DecodeArgs* args, int P, cudaStream_t stream)
{
    if (P < 1 || P > kDecMaxProj) return cudaErrorInvalidValue;
    const int num_sms = args[0].num_sms;
    long long rows_total = 0;
    for (int p = 0; p < P; ++p) rows_total += args[p].d_out;
    int count[kDecMaxProj], given = 0;
    for (int p = 0; p < P; ++p) {
        int c = (int)((long long)num_sms * args[p].d_out / rows_total);
        const int cap = (args[p].d_out + 1) / 2;
        c = c < 1 ? 1 : (c > cap ? cap : c);
        count[p] = c;
        given += c;
    }
    // what the rounding left over goes, one CTA at a time, to the projection with the most rows per CTA
    while (given < num_sms) {
        int best = -1;
        double worst = 0.0;
        for (int p = 0; p < P; ++p) {
            const double load = (double)args[p].d_out / count[p];
            if (count[p] < (args[p].d_out + 1) / 2 && load > worst) { worst = load; best = p; }
        }
        if (best < 0) break;
        ++count[best];
        ++given;
    }
    while (given > num_sms) {   // (more projections than SMs cannot happen with P <= 4; kept for safety)
        int best = 0;
        for (int p = 1; p < P; ++p) if (count[p] > count[best]) best = p;
        if (count[best] <= 1) break;
        --count[best];
        --given;
    }
    DecLaunch<kDecMaxProj> prm;
    int begin = 0, rows_per_cta = 0, max_T = 0, ntables = 0;
    bool adapters = false;
    const Arena* seen[kDecMaxTables];
    int uses[kDecMaxTables];
    // A table that serves several parts of the launch (the bindings of a dual call, the blocks of a batch of more than 16
    // tokens) gives each of them an exchange block of its own
    for (int p = 0; p < P; ++p) {
        int ti = 0;
        while (ti < ntables && seen[ti] != ars[p]) ++ti;
        if (ti == ntables) {
            if (ntables == kDecMaxTables) return cudaErrorInvalidValue;
            seen[ntables] = ars[p]; uses[ntables] = 0; prm.snap[ntables] = snaps[p];
            ++ntables;
        }
        fill_proj(prm.proj[p], *ars[p], args[p]);
        prm.proj[p].snap_idx = ti;
        if (!args[p].exch) {
            prm.proj[p].u = ars[p]->dec_u + (size_t)uses[ti] * kDecExchStride;
            prm.proj[p].sync_words = reinterpret_cast<unsigned int*>(prm.proj[p].u + kDecExchEntries);
        }
        ++uses[ti];
        prm.proj[p].cta_begin = begin; prm.proj[p].cta_count = count[p];
        begin += count[p];
        const int r = (args[p].d_out + count[p] - 1) / count[p];
        rows_per_cta = r > rows_per_cta ? r : rows_per_cta;
        max_T = args[p].T > max_T ? args[p].T : max_T;
        adapters = adapters || args[p].G > 0;
    }
    for (int t = ntables; t < kDecMaxTables; ++t) prm.snap[t] = prm.snap[0];
    for (int p = P; p < kDecMaxProj; ++p) { prm.proj[p] = prm.proj[0]; prm.proj[p].cta_begin = begin; prm.proj[p].cta_count = 0; }
    prm.x = (const __nv_bfloat16*)args[0].x;
    prm.T = max_T; prm.K = args[0].d_in; prm.P = P; prm.patience = g_dec_patience;
    return launch_decode_grid<kDecMaxProj>(prm, begin, rows_per_cta, adapters, max_T, stream);
}

}  // namespace lml
