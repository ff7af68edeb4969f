// Prefill path: y = bf16( x.W0^T + sum over pieces u_piece.B_slot^T ) on the sm_100a tensor cores.
//
// One persistent CTA per SM, 6 warps:
//   warp 0   TMA producer: streams 128x64 tiles of x and BNx64 tiles of W0 (128-byte swizzle) into
//            a ring of shared-memory stages; after the last k-block of a tile it appends one
//            stage per LoRA piece of that tile: the piece's 128x64 block of u and the BNx64 block
//            of the slot's packed B.  So the LoRA expand is just more K for the same accumulator:
//            [x | u_1 | u_2 ...] . [W0 ; B_s1 ; B_s2 ...].
//   warp 1   MMA issuer: one lane issues tcgen05.mma (M=128, N=BN, K=16) per 16 columns of a stage
//            into one of two TMEM accumulators and commits to the stage's "empty" barrier.
//   warps 2-5 epilogue: tcgen05.ld the accumulator (each warp its 32 TMEM lanes = 32 rows), round to
//            bf16 once, stage 32x32 chunks in shared memory and write them with TMA stores (or
//            row-scattered 16-byte stores when a perm is given).  Runs one tile behind the MMA
//            warp thanks to the second accumulator.
// Dual form (two slot bindings of the same segments, two outputs): the base product is computed once.
// The epilogue reads the first output out of the accumulator and tells the MMA thread; that thread
// then adds (second binding's delta - first binding's delta) on top, as further K-steps whose u
// operands come from two more sets of u blocks (second slots; first slots negated), and the epilogue
// reads the second output.  The producer slips those stages into the middle of the next tile's
// k-blocks, by when the first read is long done.
// Fused shrink (the plain call): no shrink kernel runs before this one.  The CTAs at the end of the grid, which
// own the fewest output tiles, first compute u = scale * x.A^T for a row tile each, as 128 x 64 tcgen05 products
// (x k-blocks against the A k-blocks of the segments that touch the tile, side by side in an accumulator), write
// the u blocks and raise the row tile's flag in the table's device memory; a producer waits for that flag (a
// bounded wait) before it loads the tile's u blocks.  The table's epoch, advanced by the last CTA of every such
// call, tells this call's flags from the last call's.
// For few tokens (tiles far fewer than SMs) a split-K variant follows below: a cluster of CTAs shares a
// tile and exchanges partial sums through distributed shared memory; it also has a shrink mode.
// Every wait is bounded; on give-up the CTA sets LML_FLAG_TIMEOUT, drains and frees its TMEM.
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "lml_internal.cuh"
#include "lml_ptx_sm100.cuh"

namespace lml {

using namespace ptx;

constexpr int kBM = kTileM;   // 128
constexpr int kBK = 64;       // bf16 elements per 128-byte swizzled row
constexpr int kGemmThreads = 192;
constexpr int kSegCache = 256;            // segments cached in shared memory
constexpr int kEpiChunkCols = 32;
constexpr int kEpiBufBytes = 32 * kEpiChunkCols * 2;   // 2 KB: 32 rows x 64 B

template <int BN> struct GemmCfg {
    static constexpr int kABytes = kBM * kBK * 2;
    static constexpr int kBBytes = BN * kBK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int kEpiBytes = 4 * 2 * kEpiBufBytes;
    static constexpr int kTmemCols = 2 * BN;
    static constexpr int kCtrlBytes = 256 + (kSegCache + 1) * 4 + 2 * kSegCache + 512 + 1040;   // barriers + segment cache (two slot arrays) + shrink plan + its per-tile table
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kEpiBytes + ((kCtrlBytes + 15) & ~15);
};

struct GemmCtrl {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t tmem_read1[2];   // dual form: the first output of the tile has been read out of the accumulator
    uint32_t tmem_base;
    int abort;
    uint32_t stage_info[8];   // written by the producer: k-steps (0..4) | kStage* flags
    int32_t piece[4];         // shrink form of the split-K kernel: found, slot, first row, end row of the CTA's piece
    int32_t pad[2];
};
// stage_info flags
constexpr uint32_t kStageCommit = 0x100u;   // after this stage the accumulator holds an output: commit it to the epilogue
constexpr uint32_t kStageAcc1 = 0x200u;     // the stage belongs to accumulator 1 (else 0)
constexpr uint32_t kStageFresh = 0x400u;    // first stage of a tile: wait for the accumulator to be free, overwrite it
constexpr uint32_t kStageDelta = 0x800u;    // dual form: first stage of a tile's second output: wait until the first was read

static_assert(sizeof(GemmCtrl) <= 256, "control block");
constexpr uint32_t kStageBoth = 0x2000u;    // split-K dual form: the stage's product goes into both bindings' accumulators
constexpr uint32_t kStageShrink = 0x1000u;  // a stage of a shrink pass: x tile and bits 16..18 blocks of A; as many 128 x 64 products

// Fused shrink (the plain call on whole-K tiles): the CTAs at the end of the grid, which own one tile fewer than
// the others or none more, first compute u = scale * x.A^T for a row tile each: one pass multiplies the tile's x
// k-blocks with the A blocks of up to BN / 64 segments that touch the tile (128 x 64 tcgen05 products side by side
// in an accumulator), its epilogue writes the u blocks and raises the tile's flag in the table's device memory.
constexpr int kShrMaxPasses = 8;
constexpr int kFuseTilesInKernel = 512;   // row tiles of a call whose shrink runs inside the kernel (the per-tile table in shared memory)
struct ShrPass {
    int32_t m;          // row tile
    int32_t n;          // pieces in this pass
    int32_t flag;       // the pass's number among all passes of the call: the flag it raises
    int32_t g[4];       // segment of each piece
    int32_t slot[4];
};
struct ShrPlan {
    int32_t npass;
    int32_t lora_ok;
    int32_t epoch;
    int32_t pad;
    ShrPass pass[kShrMaxPasses];
};
static_assert(sizeof(ShrPlan) <= 512, "shrink plan");

struct GemmParams {
    const int32_t* seg_offsets;
    const int32_t* slot_ids;
    const int32_t* perm;
    const int32_t* tile_identity;   // perm form: tiles whose rows stayed in place (read tmap_x0, store with TMA)
    const PlanWord* plan;
    const int32_t* slot_ids2;   // dual form: the second slot per segment (else null)
    __nv_bfloat16* y2;          // dual form: the second output
    int u_set_rows;             // dual form: rows between the three sets of u blocks (first slots, second slots, minus first)
    __nv_bfloat16* y;
    uint32_t* status;
    int T, K, N, G;
    int num_m, num_n;
    int fused;                  // the shrink runs inside this kernel (else a shrink kernel ran before it)
    int32_t* tile_flags;        // fused: [row tile] = epoch + 1 once the tile's u blocks are written
    uint32_t* fuse_sync;        // fused: [0] the table's epoch, [1] CTAs that have finished (the last one advances the epoch)
    __nv_bfloat16* u_out;       // fused: the u blocks, for writing
};

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1) lora_gemm_sm100_kernel(
    const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_x0,
    const __grid_constant__ CUtensorMap tmap_w,
    const __grid_constant__ CUtensorMap tmap_u, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_y2,
    const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ SlotSnapshot snap, const GemmParams p)
{
    using Cfg = GemmCfg<BN>;
    // One piece to a pass: a pass with one piece moves two k-blocks per stage and takes about as long as an output
    // tile; more pieces side by side (up to BN / 64 fit an accumulator) halve that rate, and every CTA's first
    // tile would wait for the longest pass.  A row tile's pieces run on different CTAs instead.
    constexpr int kShrPerPass = 1;
    const bool dual = p.slot_ids2 != nullptr;
    extern __shared__ uint8_t smem_raw[];
    // 128-byte swizzled tiles need 1024-byte alignment
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t* tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    const uint32_t epi_addr = tiles_addr + Cfg::kStages * Cfg::kStageBytes;
    uint8_t* epi_ptr = tiles_ptr + Cfg::kStages * Cfg::kStageBytes;
    GemmCtrl* ctrl = reinterpret_cast<GemmCtrl*>(epi_ptr + Cfg::kEpiBytes);
    int32_t* seg_cache = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(ctrl) + 256);
    int8_t* slot_cache = reinterpret_cast<int8_t*>(seg_cache + kSegCache + 1);
    int8_t* slot_cache2 = slot_cache + kSegCache;   // dual form: the second slot per segment
    ShrPlan* shr = reinterpret_cast<ShrPlan*>(slot_cache2 + kSegCache);
    uint16_t* shr_base = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(shr) + 512);   // [row tile] first pass; kFuseTilesInKernel + 1 entries

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.num_m * p.num_n;
    const int num_kb = (p.K + kBK - 1) / kBK;
    const bool seg_cached = p.G <= kSegCache;

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctrl->tmem_full[a]), 1);
            mbar_init(smem_u32(&ctrl->tmem_empty[a]), 4);
            mbar_init(smem_u32(&ctrl->tmem_read1[a]), 4);
        }
        ctrl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tmap(&tmap_x0);
        prefetch_tmap(&tmap_x); prefetch_tmap(&tmap_w); prefetch_tmap(&tmap_u);
        prefetch_tmap(&tmap_b); prefetch_tmap(&tmap_y);
        if (dual) prefetch_tmap(&tmap_y2);
    }
    if (seg_cached && p.G > 0) {
        for (int g = threadIdx.x; g <= p.G; g += kGemmThreads) seg_cache[g] = __ldg(p.seg_offsets + g);
        for (int g = threadIdx.x; g < p.G; g += kGemmThreads) {
            int s = __ldg(p.slot_ids + g);
            slot_cache[g] = (int8_t)((s >= 0 && s < snap.max_slots && snap.rank[s] > 0) ? s : -1);
            if (dual) {
                const int s2 = __ldg(p.slot_ids2 + g);
                slot_cache2[g] = (int8_t)((s2 >= 0 && s2 < snap.max_slots && snap.rank[s2] > 0) ? s2 : -1);
            }
        }
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctrl->tmem_base), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile int* abort = &ctrl->abort;
    if (p.G == 0 || p.fused) {   // no shrink kernel ran before this one in the call: wait for foreign work here
        grid_dependency_wait();
        grid_launch_dependents();
    }
    if (p.fused) {
        // The segment arrays are checked here (every CTA reaches the same verdict from its own copy), and the CTA's
        // shrink passes are laid out: row tiles grid-1-blockIdx, +grid, ... (the CTAs at the end of the grid own
        // the fewest output tiles), and for each the live segments that touch it, kShrPerPass to a pass.
        int bad_off = 0, bad_slot = 0;
        for (int g = threadIdx.x; g < p.G; g += kGemmThreads) {
            const int s0 = seg_cache[g], s1 = seg_cache[g + 1];
            if (s1 < s0 || s0 < 0 || s1 > p.T) bad_off = 1;
            const int sl = __ldg(p.slot_ids + g);
            if (sl != -1 && s1 > s0 && slot_rank(snap, sl) == 0) bad_slot = 1;   // an empty segment may name anything
        }
        if (threadIdx.x == 0 && (seg_cache[0] != 0 || seg_cache[p.G] != p.T)) bad_off = 1;
        bad_off = __syncthreads_or(bad_off);
        bad_slot = __syncthreads_or(bad_slot);
        // Passes of every row tile: its live pieces, kShrPerPass to a pass (threads share the tiles out) ...
        auto live_pieces = [&](int m, int skip, int take, ShrPass* out) -> int {   // counts the tile's pieces; fills `out` with pieces skip .. skip+take-1
            const int row0 = m * kBM, row1 = min(row0 + kBM, p.T);
            int lo = 0, hi = p.G;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (seg_cache[mid + 1] > row0) hi = mid; else lo = mid + 1; }
            int c = 0;
            for (int g = lo; g < p.G && seg_cache[g] < row1; ++g) {
                const int sl = slot_cache[g];
                if (sl < 0 || min(seg_cache[g + 1], row1) <= max(seg_cache[g], row0)) continue;
                if (out && c >= skip && c < skip + take) { out->g[c - skip] = g; out->slot[c - skip] = sl; }
                ++c;
            }
            return c;
        };
        for (int m = threadIdx.x; m < p.num_m; m += kGemmThreads)
            shr_base[m + 1] = (uint16_t)(bad_off ? 0 : (live_pieces(m, 0, 0, nullptr) + kShrPerPass - 1) / kShrPerPass);
        __syncthreads();
        if (threadIdx.x == 0) {
            if (blockIdx.x == 0) {
                const unsigned f = (bad_off ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_slot ? LML_FLAG_BAD_SLOT : 0u);
                if (f) atomicOr(p.status, f);
            }
            shr->lora_ok = bad_off ? 0 : 1;
            shr->epoch = (int32_t)(*reinterpret_cast<volatile uint32_t*>(p.fuse_sync));
            // ... numbered through all row tiles (shr_base[m] = first pass of tile m); pass i is the work of CTA
            // grid-1 - (i mod grid): the CTAs at the end of the grid own the fewest output tiles, and the passes
            // of a row tile with many pieces run side by side on different CTAs
            shr_base[0] = 0;
            for (int m = 0; m < p.num_m; ++m) shr_base[m + 1] = (uint16_t)(shr_base[m] + shr_base[m + 1]);
            const int total = shr_base[p.num_m];
            int np = 0, m = 0;
            for (int i = (int)gridDim.x - 1 - (int)blockIdx.x; i < total && np < kShrMaxPasses; i += (int)gridDim.x) {
                while (shr_base[m + 1] <= i) ++m;
                ShrPass& ps = shr->pass[np++];
                ps.m = m; ps.flag = i;
                const int c = live_pieces(m, (i - shr_base[m]) * kShrPerPass, kShrPerPass, &ps);
                ps.n = min(kShrPerPass, c - (i - shr_base[m]) * kShrPerPass);
            }
            shr->npass = np;
        }
        __syncthreads();
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // Stage order.  A tile is its base k-blocks followed by one stage per LoRA piece; the last of
        // these carries kStageCommit.  In the dual form every tile has a second output, the same
        // accumulator plus (second slots' delta minus first slots' delta): its stages ("delta
        // stages": one per piece of the second slot array, one per piece of the first with the
        // negated u) can only run once the epilogue has read the first output, so they are slipped
        // into the middle of the NEXT tile's k-blocks (or follow the last tile), where the MMA thread
        // does not have to wait for that.
        if (lane == 0) {
            bool lora = false, lora_known = (p.G == 0);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            auto acquire = [&]() -> bool {
                return mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, abort);
            };
            auto advance = [&]() { if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; } };
            auto learn_lora = [&]() {
                // Everything the shrink kernel wrote (plan word, u blocks) is first touched after the
                // base k-blocks of the first tile are already in flight.
                if (!lora_known) {
                    if (p.fused) lora = shr->lora_ok != 0;
                    else {
                        grid_dependency_wait();
                        grid_launch_dependents();
                        lora = p.plan->lora_ok != 0;
                    }
                    lora_known = true;
                }
            };
            // fused shrink: the u blocks of row tile m are written by another CTA of this grid, which raises the
            // tile's flag when they are complete (bounded wait; the flag's writer runs its shrink passes first thing)
            int flag_seen_m = -1;
            auto wait_u = [&](int m) {
                if (!p.fused || m == flag_seen_m) return;
                const int want = shr->epoch + 1;
                const long long t0 = clock64();
                for (int i = shr_base[m]; i < shr_base[m + 1]; ++i)
                    while (ld_acquire_gpu_s32(p.tile_flags + i) != want) {
                        if (*abort) { ok = false; return; }
                        if (clock64() - t0 > (1ll << 31)) { *abort = 1; ok = false; return; }
                    }
                fence_proxy_async_all();   // what those CTAs wrote with ordinary stores is read by TMA from here on
                flag_seen_m = m;
            };
            // slot of segment g as far as tile rows [row0, row1) are concerned; -1 = no piece
            auto piece_slot = [&](int g, int row0, int row1, bool second) -> int {
                int s0, s1, s;
                if (seg_cached) { s0 = seg_cache[g]; s1 = seg_cache[g + 1]; s = second ? slot_cache2[g] : slot_cache[g]; }
                else {
                    s0 = __ldg(p.seg_offsets + g); s1 = __ldg(p.seg_offsets + g + 1);
                    s = __ldg((second ? p.slot_ids2 : p.slot_ids) + g);
                    if (slot_rank(snap, s) == 0) s = -1;
                }
                if (min(s1, row1) <= max(s0, row0)) return -1;
                return s;
            };
            auto segment_range = [&](int row0, int row1, int& g_first, int& g_end) {
                if (seg_cached) {
                    int lo = 0, hi = p.G;
                    while (lo < hi) { int mid = (lo + hi) >> 1; if (seg_cache[mid + 1] > row0) hi = mid; else lo = mid + 1; }
                    g_first = lo;
                    g_end = g_first;
                    while (g_end < p.G && seg_cache[g_end] < row1) ++g_end;
                } else {
                    g_first = seg_upper(p.seg_offsets, p.G, row0);
                    g_end = g_first;
                    while (g_end < p.G && __ldg(p.seg_offsets + g_end) < row1) ++g_end;
                }
            };
            // one stage per piece of a tile from one of the three sets of u blocks; `flags_first` go on the
            // first stage emitted, `flags_last` on the last; returns how many stages went out
            auto emit_pieces = [&](int m, int n, int set, bool second, uint32_t acc_flag, uint32_t flags_first,
                                   uint32_t flags_last, bool count_only) -> int {
                const int row0 = m * kBM, row1 = min(row0 + kBM, p.T);
                int g_first = 0, g_end = 0, count = 0, last_piece = -1;
                if (lora) {
                    segment_range(row0, row1, g_first, g_end);
                    for (int g = g_first; g < g_end; ++g) if (piece_slot(g, row0, row1, second) >= 0) { last_piece = g; ++count; }
                }
                if (count_only) return count;
                if (count > 0) wait_u(m);
                if (!ok) return count;
                bool first = true;
                for (int g = g_first; g < g_end && ok; ++g) {
                    const int s = piece_slot(g, row0, row1, second);
                    if (s < 0) continue;
                    ok = acquire();
                    if (!ok) break;
                    const uint32_t a_dst = tiles_addr + stage * Cfg::kStageBytes;
                    const uint32_t bar = smem_u32(&ctrl->full[stage]);
                    const uint32_t ksteps = (uint32_t)((snap.rank[s] + 15) >> 4);
                    ctrl->stage_info[stage] = ksteps | acc_flag | (first ? flags_first : 0u) | (g == last_piece ? flags_last : 0u);
                    first = false;
                    mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                    tma_load_2d(a_dst, &tmap_u, bar, 0, set * p.u_set_rows + (m + g) * kBM);
                    tma_load_3d(a_dst + Cfg::kABytes, &tmap_b, bar, 0, n * BN, s);
                    advance();
                }
                return count;
            };
            // a stage without operands: only its flags matter to the MMA thread
            auto emit_marker = [&](uint32_t info) {
                ok = acquire();
                if (!ok) return;
                ctrl->stage_info[stage] = info;
                mbar_arrive(smem_u32(&ctrl->full[stage]));
                advance();
            };
            // the delta stages of tile (m, n) on accumulator flag acc_flag
            auto emit_delta = [&](int m, int n, uint32_t acc_flag) {
                const int n_new = emit_pieces(m, n, 1, true, acc_flag, 0u, 0u, true);
                const int n_old = emit_pieces(m, n, 2, false, acc_flag, 0u, 0u, true);
                if (n_new + n_old == 0) { emit_marker(acc_flag | kStageDelta | kStageCommit); return; }
                emit_pieces(m, n, 1, true, acc_flag, kStageDelta, n_old == 0 ? kStageCommit : 0u, false);
                if (ok && n_old > 0) emit_pieces(m, n, 2, false, acc_flag, n_new == 0 ? kStageDelta : 0u, kStageCommit, false);
            };
            int ordinal = 0, prev_m = -1, prev_n = -1;
            // this CTA's shrink passes: a pass is num_kb stages of [x k-block | A k-blocks of its pieces]
            for (int ps = 0; p.fused && ps < shr->npass && ok; ++ps, ++ordinal) {
                const ShrPass& sp = shr->pass[ps];
                const uint32_t acc_flag = (ordinal & 1) ? kStageAcc1 : 0u;
                const bool in_place = p.tile_identity && __ldg(p.tile_identity + sp.m);
                // (a pass with one piece moves 24 KB per k-block: two k-blocks share a stage, so that as many bytes
                // are on their way as in the tiles' stages)
                const int sub_bytes = Cfg::kABytes + sp.n * (64 * kBK * 2);
                const int per_stage = 2 * sub_bytes <= Cfg::kStageBytes ? 2 : 1;
                for (int kb = 0; kb < num_kb && ok; kb += per_stage) {
                    ok = acquire();
                    if (!ok) break;
                    const int nsub = min(per_stage, num_kb - kb);
                    const uint32_t bar = smem_u32(&ctrl->full[stage]);
                    ctrl->stage_info[stage] = 4u | acc_flag | kStageShrink | ((uint32_t)sp.n << 16) | ((uint32_t)nsub << 20) |
                                              (kb == 0 ? kStageFresh : 0u) | (kb + nsub >= num_kb ? kStageCommit : 0u);
                    mbar_arrive_expect_tx(bar, (uint32_t)(nsub * sub_bytes));
                    for (int j = 0; j < nsub; ++j) {
                        const uint32_t a_dst = tiles_addr + stage * Cfg::kStageBytes + j * sub_bytes;
                        if (in_place) tma_load_2d(a_dst, &tmap_x0, bar, (kb + j) * kBK, sp.m * kBM);
                        else tma_load_2d(a_dst, &tmap_x, bar, (kb + j) * kBK, sp.m * kBM);
                        for (int i = 0; i < sp.n; ++i)
                            tma_load_3d(a_dst + Cfg::kABytes + i * (64 * kBK * 2), &tmap_a, bar, (kb + j) * kBK, 0, sp.slot[i]);
                    }
                    advance();
                }
            }
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++ordinal) {
                const int m = tile % p.num_m, n = tile / p.num_m;
                const int row0 = m * kBM;
                const uint32_t acc_flag = (ordinal & 1) ? kStageAcc1 : 0u;
                const bool in_place = p.tile_identity && __ldg(p.tile_identity + m);   // rows of x never copied
                int pieces = 0;
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    if (kb == num_kb - 1) {
                        learn_lora();
                        pieces = emit_pieces(m, n, 0, false, acc_flag, 0u, 0u, true);
                    }
                    if (dual && prev_m >= 0 && kb == min((num_kb + 1) / 2, num_kb - 1)) {
                        learn_lora();
                        emit_delta(prev_m, prev_n, acc_flag ^ kStageAcc1);
                        if (!ok) break;
                    }
                    ok = acquire();
                    if (!ok) break;
                    const uint32_t a_dst = tiles_addr + stage * Cfg::kStageBytes;
                    const uint32_t bar = smem_u32(&ctrl->full[stage]);
                    ctrl->stage_info[stage] = 4u | acc_flag | (kb == 0 ? kStageFresh : 0u) |
                                              ((kb == num_kb - 1 && pieces == 0) ? kStageCommit : 0u);
                    mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                    // two call sites on purpose: each names its tensor map as a kernel-parameter constant
                    if (in_place) tma_load_2d(a_dst, &tmap_x0, bar, kb * kBK, row0);
                    else tma_load_2d(a_dst, &tmap_x, bar, kb * kBK, row0);
                    tma_load_2d(a_dst + Cfg::kABytes, &tmap_w, bar, kb * kBK, n * BN);
                    advance();
                }
                if (ok && pieces > 0) emit_pieces(m, n, 0, false, acc_flag, 0u, kStageCommit, false);
                prev_m = m; prev_n = n;
            }
            if (ok && dual && prev_m >= 0) {
                learn_lora();
                emit_delta(prev_m, prev_n, ((ordinal - 1) & 1) ? kStageAcc1 : 0u);
            }
            // Leave only after every load issued above has landed (its stage was consumed or its
            // full barrier completed): wait for the ring to drain.
            for (int i = 0; i < Cfg::kStages && ok; ++i) { ok = acquire(); advance(); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Walks the same schedule as the producer.  The base k-blocks are always four K-steps and need no
        // side-band word; the last one, the LoRA stages after it and the delta stages carry one (how
        // many K-steps, and whether an output is complete after the stage).
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t empty_ph0 = 0, empty_ph1 = 0, read1_ph0 = 0, read1_ph1 = 0;
            bool ok = true;
            // one stage: ksteps MMAs into d_tmem, then the stage goes back to the producer
            auto issue = [&](uint32_t d_tmem, int ksteps, uint32_t& accumulate) {
                const uint32_t a_addr = tiles_addr + stage * Cfg::kStageBytes;
                const uint64_t adesc = umma_desc_k128(a_addr);
                const uint64_t bdesc = umma_desc_k128(a_addr + Cfg::kABytes);
#pragma unroll 4
                for (int k = 0; k < ksteps; ++k) {
                    // 16 bf16 columns = 32 bytes further along the swizzled row: +2 in 16-byte units
                    umma_bf16(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, accumulate);
                    accumulate = 1;
                }
                umma_commit(smem_u32(&ctrl->empty[stage]));
                if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
            };
            // stages with a side-band word, up to and including the one that completes an output
            auto flagged_stages = [&](int acc, uint32_t& accumulate) {
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (bool more = true; more && ok;) {
                    ok = mbar_wait(smem_u32(&ctrl->full[stage]), phase, abort);
                    if (!ok) break;
                    const uint32_t info = ctrl->stage_info[stage];
                    more = (info & kStageCommit) == 0;
                    issue(d_tmem, (int)(info & 0xffu), accumulate);
                }
                if (ok) umma_commit(smem_u32(&ctrl->tmem_full[acc]));
            };
            // the second output of the tile that sits in accumulator acc: once the epilogue has read the
            // first, add (second slots' delta - first slots' delta) on top
            auto delta_stages = [&](int acc) {
                uint32_t& ph = acc ? read1_ph1 : read1_ph0;
                ok = mbar_wait(smem_u32(&ctrl->tmem_read1[acc]), ph, abort);
                if (!ok) return;
                ph ^= 1u;
                tc_fence_after();
                uint32_t accumulate = 1;
                flagged_stages(acc, accumulate);
            };
            int ordinal = 0;
            // this CTA's shrink passes: per stage, one 128 x 64 product per piece, side by side in the accumulator
            for (int ps = 0; p.fused && ps < shr->npass && ok; ++ps, ++ordinal) {
                constexpr uint32_t idesc64 = umma_idesc_bf16(kBM, 64);
                const int acc = ordinal & 1;
                uint32_t& eph = acc ? empty_ph1 : empty_ph0;
                ok = mbar_wait(smem_u32(&ctrl->tmem_empty[acc]), eph ^ 1u, abort);
                if (!ok) break;
                eph ^= 1u;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                bool fresh = true;
                for (bool more = true; more && ok;) {
                    ok = mbar_wait(smem_u32(&ctrl->full[stage]), phase, abort);
                    if (!ok) break;
                    const uint32_t info = ctrl->stage_info[stage];
                    more = (info & kStageCommit) == 0;
                    const int npc = (int)((info >> 16) & 7u), nsub = (int)((info >> 20) & 3u);
                    const int sub_bytes = Cfg::kABytes + npc * (64 * kBK * 2);
                    tc_fence_after();
                    for (int j = 0; j < nsub; ++j) {
                        const uint32_t a_addr = tiles_addr + stage * Cfg::kStageBytes + j * sub_bytes;
                        const uint64_t adesc = umma_desc_k128(a_addr);
                        for (int i = 0; i < npc; ++i) {
                            const uint64_t bdesc = umma_desc_k128(a_addr + Cfg::kABytes + i * (64 * kBK * 2));
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_bf16(d_tmem + (uint32_t)(64 * i), adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc64,
                                          (!fresh || k > 0) ? 1u : 0u);
                        }
                        fresh = false;
                    }
                    umma_commit(smem_u32(&ctrl->empty[stage]));
                    if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&ctrl->tmem_full[acc]));
            }
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++ordinal) {
                const int acc = ordinal & 1;
                uint32_t& eph = acc ? empty_ph1 : empty_ph0;
                ok = mbar_wait(smem_u32(&ctrl->tmem_empty[acc]), eph ^ 1u, abort);
                if (!ok) break;
                eph ^= 1u;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                uint32_t accumulate = 0;
                const int mid = min((num_kb + 1) / 2, num_kb - 1);
                for (int kb = 0; kb < num_kb - 1 && ok; ++kb) {
                    if (dual && ordinal > 0 && kb == mid) { delta_stages(acc ^ 1); if (!ok) break; }
                    ok = mbar_wait(smem_u32(&ctrl->full[stage]), phase, abort);
                    if (!ok) break;
                    issue(d_tmem, 4, accumulate);
                }
                if (!ok) break;
                if (dual && ordinal > 0 && mid == num_kb - 1) { delta_stages(acc ^ 1); if (!ok) break; }
                flagged_stages(acc, accumulate);   // the last k-block and the tile's LoRA pieces
            }
            if (ok && dual && ordinal > 0) delta_stages((ordinal - 1) & 1);
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int ew = warp - 2;
        const uint32_t buf_addr0 = epi_addr + (uint32_t)(ew * 2 * kEpiBufBytes);
        uint8_t* buf_ptr0 = epi_ptr + ew * 2 * kEpiBufBytes;
        int acc = 0;
        uint32_t full_ph0 = 0, full_ph1 = 0;
        int buf = 0;
        bool ok = true;
        // this CTA's shrink passes: scale, zero the rows outside the segment, round, write the u blocks; after a
        // tile's last pass its flag goes up (release: the four warps' stores are complete)
        for (int ps = 0; p.fused && ps < shr->npass && ok; ++ps) {
            const ShrPass& sp = shr->pass[ps];
            uint32_t& fph = acc ? full_ph1 : full_ph0;
            ok = mbar_wait_warp(smem_u32(&ctrl->tmem_full[acc]), fph, abort);
            if (!ok) break;
            fph ^= 1u;
            tc_fence_after();
            const int pos = sp.m * kBM + q * 32 + lane;
            const int row0 = sp.m * kBM, row1 = min(row0 + kBM, p.T);
            for (int i = 0; i < sp.n; ++i) {
                const int g = sp.g[i];
                const bool mine = pos >= max(seg_cache[g], row0) && pos < min(seg_cache[g + 1], row1);
                const float sc = mine ? snap.scale[sp.slot[i]] : 0.f;
                __nv_bfloat16* out = p.u_out + ((size_t)(sp.m + g) * kBM + q * 32 + lane) * kRankPad;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + 64 * i + 32 * c), r);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[8 * j + 0]) * sc, __uint_as_float(r[8 * j + 1]) * sc);
                        v.y = pack_bf16(__uint_as_float(r[8 * j + 2]) * sc, __uint_as_float(r[8 * j + 3]) * sc);
                        v.z = pack_bf16(__uint_as_float(r[8 * j + 4]) * sc, __uint_as_float(r[8 * j + 5]) * sc);
                        v.w = pack_bf16(__uint_as_float(r[8 * j + 6]) * sc, __uint_as_float(r[8 * j + 7]) * sc);
                        if (!mine) v = make_uint4(0, 0, 0, 0);   // (0 * garbage may be a NaN)
                        *reinterpret_cast<uint4*>(out + c * 32 + j * 8) = v;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[acc]));
            fence_proxy_async_all();   // the blocks will be read by TMA
            __threadfence();
            asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps
            if (warp == 2 && lane == 0) st_release_gpu_s32(p.tile_flags + sp.flag, shr->epoch + 1);
            acc ^= 1;
        }
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int m = tile % p.num_m, n = tile / p.num_m;
            const int row_base = m * kBM + q * 32;
            const bool scatter = p.perm != nullptr && !(p.tile_identity && __ldg(p.tile_identity + m));
            for (int pass = 0; pass < (dual ? 2 : 1) && ok; ++pass) {
                uint32_t& fph = acc ? full_ph1 : full_ph0;
                ok = mbar_wait_warp(smem_u32(&ctrl->tmem_full[acc]), fph, abort);
                if (!ok) break;
                fph ^= 1u;
                tc_fence_after();
                const bool last_pass = pass == (dual ? 1 : 0);
                __nv_bfloat16* yout = pass == 0 ? p.y : p.y2;
                const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
                for (int c = 0; c < BN / kEpiChunkCols; ++c) {
                    uint32_t r[32];
                    tmem_ld_32x32(t_addr + (uint32_t)(c * kEpiChunkCols), r);
                    tmem_ld_wait();
                    if (c == BN / kEpiChunkCols - 1) {
                        // accumulator fully read: hand it back to the MMA warp (for the tile's second
                        // output, or for the next tile)
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(last_pass ? &ctrl->tmem_empty[acc] : &ctrl->tmem_read1[acc]));
                    }
                    const int col0 = n * BN + c * kEpiChunkCols;
                    if (col0 >= p.N || row_base >= p.T) continue;   // nothing of this chunk is inside y
                    // the buffer we are about to overwrite must have been read by its earlier store
                    if (lane == 0) tma_store_wait_read<1>();
                    __syncwarp();
                    uint8_t* bp = buf_ptr0 + buf * kEpiBufBytes;
                    const uint32_t ba = buf_addr0 + (uint32_t)(buf * kEpiBufBytes);
                    // row = lane: 64 bytes, four 16-byte chunks, 64-byte swizzle (chunk ^= (row >> 1) & 3)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(r[8 * j + 0]), __uint_as_float(r[8 * j + 1]));
                        v.y = pack_bf16(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3]));
                        v.z = pack_bf16(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5]));
                        v.w = pack_bf16(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7]));
                        const int phys = j ^ ((lane >> 1) & 3);
                        *reinterpret_cast<uint4*>(bp + lane * 64 + phys * 16) = v;
                    }
                    if (!scatter) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            // two call sites on purpose: each names its tensor map as a kernel-parameter constant
                            if (pass == 0) tma_store_2d(&tmap_y, ba, col0, row_base);
                            else tma_store_2d(&tmap_y2, ba, col0, row_base);
                            tma_store_commit();
                        }
                    } else {
                        __syncwarp();
                        // scatter: 4 lanes write one 64-byte row piece; 8 rows per pass
#pragma unroll
                        for (int sp = 0; sp < 4; ++sp) {
                            const int rr = sp * 8 + (lane >> 2), j = lane & 3;
                            const int pos = row_base + rr;
                            if (pos < p.T && col0 + j * 8 < p.N) {
                                const int row = __ldg(p.perm + pos);
                                if (row >= 0 && row < p.T) {
                                    const int phys = j ^ ((rr >> 1) & 3);
                                    uint4 v = *reinterpret_cast<const uint4*>(bp + rr * 64 + phys * 16);
                                    *reinterpret_cast<uint4*>(yout + (size_t)row * p.N + col0 + j * 8) = v;
                                }
                            }
                        }
                        __syncwarp();
                    }
                    buf ^= 1;
                }
            }
            acc ^= 1;
        }
        if (lane == 0) tma_store_wait_all();
    }

    __syncthreads();
    if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.status, LML_FLAG_TIMEOUT);
    if (threadIdx.x == 0 && p.fused) {
        // the last CTA to finish moves the table's epoch on: the flags of this call mean nothing to the next one
        __threadfence();
        if (atomicAdd(p.fuse_sync + 1, 1u) == gridDim.x - 1) {
            p.fuse_sync[1] = 0u;
            p.fuse_sync[0] = (uint32_t)(shr->epoch + 1);
        }
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// ---- split-K variant for few tokens ---------------------------------------------------------------------
// With a few hundred tokens or fewer the layer is bound by the read of W0, and 128 x 256 tiles give far
// fewer CTAs than the machine has SMs.  Here a cluster of S CTAs shares one tile: CTA r multiplies its
// share of the k-blocks (and of the tile's LoRA pieces, which are just more K) into its own TMEM
// accumulator, so S times as many SMs stream W0.  The partial sums are then exchanged through
// distributed shared memory: the tile's eight 32-column chunks are dealt out to the CTAs, every CTA
// writes each chunk of its partial sums into the owner's (by then idle) stage memory, and the owner adds
// the S contributions in rank order, rounds once and writes its columns of y.  Two cluster barriers
// frame the exchange: nobody writes into a CTA that is still multiplying, nobody adds before all
// have written.  Warp roles and the stage ring are those of the kernel above; every stage carries its
// side-band word.
constexpr int kSplitMaxS = 8;

__device__ __forceinline__ void st_shared_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1) lora_gemm_sm100_splitk_kernel(
    const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_x0,
    const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_u,
    const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ SlotSnapshot snap, const GemmParams p)
{
    using Cfg = GemmCfg<BN>;
    constexpr int kSplitChunks = BN / kEpiChunkCols;   // 32-column chunks of the tile: 4 or 8
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t* tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    uint8_t* epi_ptr = tiles_ptr + Cfg::kStages * Cfg::kStageBytes;
    GemmCtrl* ctrl = reinterpret_cast<GemmCtrl*>(epi_ptr + Cfg::kEpiBytes);
    int32_t* seg_cache = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(ctrl) + 256);
    int8_t* slot_cache = reinterpret_cast<int8_t*>(seg_cache + kSegCache + 1);
    int8_t* slot_cache2 = slot_cache + kSegCache;   // dual form: the second slot per segment
    // Dual form (two bindings of the same segments, two outputs): the k-blocks pass through shared memory once and
    // are multiplied into two accumulators (with few tokens the tensor cores have time to spare: the kernel is
    // bound by the read of W0); each binding's pieces go to its own accumulator, and the exchange runs twice.
    const bool dual = p.slot_ids2 != nullptr;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = (int)gridDim.x, rank = (int)blockIdx.x;   // the cluster spans the grid's x dimension
    const int n = (int)blockIdx.y;
    const int m = (int)blockIdx.z;
    const int num_kb = (p.K + kBK - 1) / kBK;
    const bool seg_cached = p.G <= kSegCache;
    // chunks of the tile's 256 columns that CTA r reduces: [first(r), first(r + 1))
    auto first_chunk = [&](int r) { return r * kSplitChunks / S; };
    const int cpr = (kSplitChunks + S - 1) / S;   // most chunks any CTA owns

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctrl->tmem_full[0]), 1);
        ctrl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tmap(&tmap_x0); prefetch_tmap(&tmap_x); prefetch_tmap(&tmap_w); prefetch_tmap(&tmap_u); prefetch_tmap(&tmap_b);
    }
    if (seg_cached && p.G > 0) {
        for (int g = threadIdx.x; g <= p.G; g += kGemmThreads) seg_cache[g] = __ldg(p.seg_offsets + g);
        for (int g = threadIdx.x; g < p.G; g += kGemmThreads) {
            int s = __ldg(p.slot_ids + g);
            slot_cache[g] = (int8_t)((s >= 0 && s < snap.max_slots && snap.rank[s] > 0) ? s : -1);
            if (dual) {
                const int s2 = __ldg(p.slot_ids2 + g);
                slot_cache2[g] = (int8_t)((s2 >= 0 && s2 < snap.max_slots && snap.rank[s2] > 0) ? s2 : -1);
            }
        }
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctrl->tmem_base), dual ? 2 * BN : BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile int* abort = &ctrl->abort;
    if (p.G == 0) {   // no shrink kernel ran before this one in the call: wait for foreign work here
        grid_dependency_wait();
        grid_launch_dependents();
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            auto acquire = [&]() -> bool { return mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, abort); };
            auto advance = [&]() { if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; } };
            const int row0 = m * kBM, row1 = min(row0 + kBM, p.T);
            const bool in_place = p.tile_identity && __ldg(p.tile_identity + m);
            const int kb0 = rank * num_kb / S, kb1 = (rank + 1) * num_kb / S;
            auto piece_slot = [&](int g, bool second) -> int {
                int s0, s1, s;
                if (seg_cached) { s0 = seg_cache[g]; s1 = seg_cache[g + 1]; s = second ? slot_cache2[g] : slot_cache[g]; }
                else {
                    s0 = __ldg(p.seg_offsets + g); s1 = __ldg(p.seg_offsets + g + 1);
                    s = __ldg((second ? p.slot_ids2 : p.slot_ids) + g);
                    if (slot_rank(snap, s) == 0) s = -1;
                }
                return min(s1, row1) <= max(s0, row0) ? -1 : s;
            };
            // base k-blocks first: they do not depend on the shrink kernel that precedes this one
            for (int kb = kb0; kb < kb1 && ok; ++kb) {
                ok = acquire();
                if (!ok) break;
                const uint32_t a_dst = tiles_addr + stage * Cfg::kStageBytes;
                const uint32_t bar = smem_u32(&ctrl->full[stage]);
                ctrl->stage_info[stage] = 4u | (dual ? kStageBoth : 0u);
                mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                if (in_place) tma_load_2d(a_dst, &tmap_x0, bar, kb * kBK, row0);
                else tma_load_2d(a_dst, &tmap_x, bar, kb * kBK, row0);
                tma_load_2d(a_dst + Cfg::kABytes, &tmap_w, bar, kb * kBK, n * BN);
                advance();
            }
            // this CTA's share of the tile's LoRA pieces
            bool lora = false;
            if (p.G > 0) {
                grid_dependency_wait();
                grid_launch_dependents();
                lora = p.plan->lora_ok != 0;
            }
            if (lora && ok) {
                int g_first, g_end;
                if (seg_cached) {
                    int lo = 0, hi = p.G;
                    while (lo < hi) { int mid = (lo + hi) >> 1; if (seg_cache[mid + 1] > row0) hi = mid; else lo = mid + 1; }
                    g_first = lo;
                    g_end = g_first;
                    while (g_end < p.G && seg_cache[g_end] < row1) ++g_end;
                } else {
                    g_first = seg_upper(p.seg_offsets, p.G, row0);
                    g_end = g_first;
                    while (g_end < p.G && __ldg(p.seg_offsets + g_end) < row1) ++g_end;
                }
                // segment g's piece goes to CTA g mod S: which CTA adds a row's LoRA term depends only on the
                // row's own segment, so a row's bits do not change with what other segments are bound to
                for (int side = 0; side < (dual ? 2 : 1) && ok; ++side)
                    for (int g = g_first; g < g_end && ok; ++g) {
                        if (g % S != rank) continue;
                        const int s = piece_slot(g, side == 1);
                        if (s < 0) continue;
                        ok = acquire();
                        if (!ok) break;
                        const uint32_t a_dst = tiles_addr + stage * Cfg::kStageBytes;
                        const uint32_t bar = smem_u32(&ctrl->full[stage]);
                        ctrl->stage_info[stage] = (uint32_t)((snap.rank[s] + 15) >> 4) | (side ? kStageAcc1 : 0u);
                        mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                        tma_load_2d(a_dst, &tmap_u, bar, 0, side * p.u_set_rows + (m + g) * kBM);   // (the second binding's u blocks: the second set)
                        tma_load_3d(a_dst + Cfg::kABytes, &tmap_b, bar, 0, n * BN, s);
                        advance();
                    }
            }
            if (ok) {   // end of this CTA's K: a stage without operands
                ok = acquire();
                if (ok) {
                    ctrl->stage_info[stage] = kStageCommit;
                    mbar_arrive(smem_u32(&ctrl->full[stage]));
                    advance();
                }
            }
            // leave the role only after every load has landed and been consumed
            for (int i = 0; i < Cfg::kStages && ok; ++i) { ok = acquire(); advance(); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN);
            int stage = 0;
            uint32_t phase = 0, accumulate = 0, accumulate2 = 0;
            bool ok = true;
            for (bool more = true; more && ok;) {
                ok = mbar_wait(smem_u32(&ctrl->full[stage]), phase, abort);
                if (!ok) break;
                const uint32_t info = ctrl->stage_info[stage];
                more = (info & kStageCommit) == 0;
                const int ksteps = (int)(info & 0xffu);
                const uint32_t a_addr = tiles_addr + stage * Cfg::kStageBytes;
                const uint64_t adesc = umma_desc_k128(a_addr);
                const uint64_t bdesc = umma_desc_k128(a_addr + Cfg::kABytes);
                tc_fence_after();
                if ((info & kStageAcc1) == 0) {
#pragma unroll 4
                    for (int k = 0; k < ksteps; ++k) {
                        umma_bf16(tmem_base, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, accumulate);
                        accumulate = 1;
                    }
                }
                if (info & (kStageAcc1 | kStageBoth)) {   // the second binding's accumulator
#pragma unroll 4
                    for (int k = 0; k < ksteps; ++k) {
                        umma_bf16(tmem_base + (uint32_t)BN, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, accumulate2);
                        accumulate2 = 1;
                    }
                }
                umma_commit(smem_u32(&ctrl->empty[stage]));
                if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit(smem_u32(&ctrl->tmem_full[0]));
            ctrl->pad[0] = (int32_t)accumulate;    // 0: this CTA had no K at all, its accumulator holds nothing
            ctrl->pad[1] = (int32_t)accumulate2;   // the same for the second binding's
        }
    }
    // ---------------------------------------------------------------------- exchange and reduction
    __syncwarp();   // (the producer's and the MMA issuer's other lanes waited here: the cluster barrier wants whole warps)
    bool ok = true;
    if (warp >= 2) {
        ok = mbar_wait_warp(smem_u32(&ctrl->tmem_full[0]), 0u, abort);   // this CTA's MMAs are complete: so are its loads
        tc_fence_after();
    }
    const int q = warp & 3;   // TMEM lane quarter an epilogue warp may read
    const int row = q * 32 + lane;
    for (int o = 0; o < (dual ? 2 : 1); ++o) {   // one exchange per output
    __nv_bfloat16* const yout = o ? p.y2 : p.y;
    cluster_sync_all();   // every CTA of the cluster is done with its stage memory (and with the exchange before this one)
    if (warp >= 2 && ok) {
        const bool have = ctrl->pad[o] != 0;
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(o * BN);
        int owner = 0;
#pragma unroll 1
        for (int c = 0; c < kSplitChunks; ++c) {
            while (first_chunk(owner + 1) <= c) ++owner;
            uint32_t r[32];
            tmem_ld_32x32(t_addr + (uint32_t)(c * kEpiChunkCols), r);
            tmem_ld_wait();
            if (!have) {
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = 0u;
            }
            // slot (this CTA's rank, chunk within the owner's share) of the owner's receive area, 16 KB: the
            // 16-byte pieces of the 128 rows, piece-major, so that a warp's store is 512 contiguous bytes
            const uint32_t local = tiles_addr + (uint32_t)((rank * cpr + (c - first_chunk(owner))) * (kBM * 128) + row * 16);
            const uint32_t remote = mapa_shared(local, (uint32_t)owner);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                st_shared_cluster_v4(remote + (uint32_t)(j * kBM * 16), r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        }
        tc_fence_before();
    }
    cluster_sync_all();   // all contributions have arrived
    if (warp >= 2 && ok) {
        const int pos = m * kBM + row;
        const bool scatter = p.perm != nullptr && !(p.tile_identity && __ldg(p.tile_identity + m));
        int out_row = pos;
        if (pos < p.T && scatter) out_row = __ldg(p.perm + pos);
        const bool row_ok = pos < p.T && out_row >= 0 && out_row < p.T;
        const int c_first = first_chunk(rank), c_end = first_chunk(rank + 1);
#pragma unroll 1
        for (int c = c_first; c < c_end; ++c) {
            float acc[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = 0.f;
            for (int src = 0; src < S; ++src) {   // rank order: the sum does not depend on timing
                const uint8_t* rp = tiles_ptr + (size_t)(src * cpr + (c - c_first)) * (kBM * 128) + row * 16;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 v = *reinterpret_cast<const float4*>(rp + j * kBM * 16);
                    acc[4 * j] += v.x; acc[4 * j + 1] += v.y; acc[4 * j + 2] += v.z; acc[4 * j + 3] += v.w;
                }
            }
            const int col0 = n * BN + c * kEpiChunkCols;
            if (!row_ok) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (col0 + j * 8 >= p.N) continue;
                uint4 v;
                v.x = pack_bf16(acc[8 * j + 0], acc[8 * j + 1]);
                v.y = pack_bf16(acc[8 * j + 2], acc[8 * j + 3]);
                v.z = pack_bf16(acc[8 * j + 4], acc[8 * j + 5]);
                v.w = pack_bf16(acc[8 * j + 6], acc[8 * j + 7]);
                *reinterpret_cast<uint4*>(yout + (size_t)out_row * p.N + col0 + j * 8) = v;
            }
        }
    }
    }   // outputs
    __syncthreads();
    if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.status, LML_FLAG_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, dual ? 2 * BN : BN);
    }
}

// ---- host side ---------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

static CUtensorMapSwizzle swizzle_for(uint32_t box_inner_elems)
{
    return box_inner_elems * 2 >= 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                      : (box_inner_elems * 2 == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

bool encode_tmap_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes,
                    uint32_t box_inner, uint32_t box_outer)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_inner), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_tmap_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                    uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    cuuint32_t box[3] = {b0, b1, b2};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(b0), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t gemm_sm100_init(int /*device*/)
{
    cudaError_t e = cudaFuncSetAttribute(lora_gemm_sm100_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         GemmCfg<256>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lora_gemm_sm100_splitk_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GemmCfg<256>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lora_gemm_sm100_splitk_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GemmCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(lora_gemm_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                GemmCfg<128>::kSmemBytes);
}

int gemm_pick_bn(int T, int d_out, int num_sms)
{
    const int num_m = (T + kBM - 1) / kBM;
    const int tiles256 = num_m * ((d_out + 255) / 256), tiles128 = num_m * ((d_out + 127) / 128);
    // Rounds of tiles over the SMs times the cost of a tile: a 128-column tile takes about 0.82 of the
    // time of a 256-column one (measured: the narrow kernel needs 1.64 times as long for the same work).
    const float t256 = (float)((tiles256 + num_sms - 1) / num_sms);
    const float t128 = 0.82f * (float)((tiles128 + num_sms - 1) / num_sms);
    return t256 <= t128 ? 256 : 128;
}

// Split-K choice for few tokens: tile width and how many CTAs share a tile (split 0: do not use it).
// It pays while the 128-column tiles are too few to keep most SMs busy.  Of the shapes whose clusters all
// fit the machine at once, take the one with the most CTAs, and among equals the smaller cluster (less
// to exchange); every CTA keeps at least two k-blocks, and the exchange area must fit the stage memory.
struct SplitChoice { int bn, split; };
// The table's override (LML_GEMM_SPLIT, read once when the table is created; a test knob): "<bn>x<split>"
// forces that shape, 0 switches the split-K kernel off.  Returns false when the variable is not set.
bool gemm_split_override(int* bn_out, int* split_out)
{
    *bn_out = -1; *split_out = -1;
    const char* e = getenv("LML_GEMM_SPLIT");
    if (!e) return false;
    int bn = 0, sp = 0;
    if (sscanf(e, "%dx%d", &bn, &sp) == 2 && (bn == 128 || bn == 256) && sp >= 2 && sp <= kSplitMaxS &&
        sp * ((bn / 32 + sp - 1) / sp) * 16384 <= GemmCfg<128>::kStages * GemmCfg<128>::kStageBytes) {
        *bn_out = bn; *split_out = sp;
    } else {
        *bn_out = 0; *split_out = 0;
    }
    return true;
}

static SplitChoice gemm_pick_split(int T, int d_in, int d_out, int num_sms, int forced_bn, int forced_split)
{
    static int max_clusters[2][kSplitMaxS + 1];
    static std::once_flag probed;
    if (forced_bn >= 0) return {forced_bn, forced_split};
    std::call_once(probed, [&]() {   // clusters of each size that can be resident together
        for (int w = 0; w < 2; ++w)
            for (int S = 2; S <= kSplitMaxS; ++S) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(S, num_sms / S, 1);
                cfg.blockDim = dim3(kGemmThreads);
                cfg.dynamicSmemBytes = w ? GemmCfg<256>::kSmemBytes : GemmCfg<128>::kSmemBytes;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
                cfg.attrs = attr; cfg.numAttrs = 1;
                int n = 0;
                cudaError_t e = w ? cudaOccupancyMaxActiveClusters(&n, lora_gemm_sm100_splitk_kernel<256>, &cfg)
                                  : cudaOccupancyMaxActiveClusters(&n, lora_gemm_sm100_splitk_kernel<128>, &cfg);
                if (e != cudaSuccess) { n = 0; (void)cudaGetLastError(); }
                max_clusters[w][S] = n;
            }
    });
    const int num_m = (T + kBM - 1) / kBM, num_kb = (d_in + kBK - 1) / kBK;
    if (num_m * ((d_out + 127) / 128) * 4 > num_sms * 3) return {0, 0};   // enough tiles without splitting
    SplitChoice best = {0, 0};
    int best_ctas = 0;
    for (int S = 2; S <= kSplitMaxS; ++S)
        for (int w = 0; w < 2; ++w) {
            const int bn = w ? 256 : 128;
            const int tiles = num_m * ((d_out + bn - 1) / bn);
            const int cpr = (bn / 32 + S - 1) / S;
            if (tiles > max_clusters[w][S] || num_kb < 2 * S) continue;
            if (S * cpr * 16384 > GemmCfg<128>::kStages * GemmCfg<128>::kStageBytes) continue;
            if (tiles * S > best_ctas) { best_ctas = tiles * S; best = {bn, S}; }
        }
    return best;
}

// Tensor maps of the caller's buffers are kept per table: a serving loop calls with the same few
// (pointer, shape) combinations over and over, and encoding a map costs a driver call each time.
bool TmapCache::get_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint64_t stride_bytes,
                       uint32_t box_inner, uint32_t box_outer)
{
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i) {
        const Key& k = keys[i];
        if (k.base == base && k.inner == inner && k.outer == outer && k.stride == stride_bytes && k.box_inner == box_inner &&
            k.box_outer == box_outer) {
            *out = maps[i];
            return true;
        }
    }
    CUtensorMap m;
    if (!encode_tmap_2d(&m, base, inner, outer, stride_bytes, box_inner, box_outer)) return false;
    const int slot = used < kEntries ? used++ : (next = (next + 1) % kEntries);
    keys[slot] = Key{base, inner, outer, stride_bytes, box_inner, box_outer};
    maps[slot] = m;
    *out = m;
    return true;
}

// Whether the shrink can run inside the GEMM kernel for this call: whole-K tiles, the segment arrays in the
// kernel's shared-memory cache, a flag per row tile in the table's array, and no CTA with more shrink passes
// than its plan holds (worst case: every segment touches every one of its row tiles).
bool gemm_can_fuse_shrink(int T, int d_in, int d_out, int G, int num_sms, int split_bn, int split_s)
{
    if (G <= 0 || G > kSegCache) return false;
    if (gemm_pick_split(T, d_in, d_out, num_sms, split_bn, split_s).split) return false;
    // A shrink pass takes about as long as an output tile, whatever its width.  It pays where some CTAs have a
    // tile's time to spare and the others do not reach their first pieces before it is over: 256-column tiles in
    // more than one wave, and few enough passes that no CTA gets two.
    if (gemm_pick_bn(T, d_out, num_sms) != 256) return false;
    const int num_m = (T + kBM - 1) / kBM, num_n = (d_out + 255) / 256;
    if (num_m > kFuseTilesInKernel || num_m * num_n <= num_sms) return false;
    const int worst_passes = num_m + G;   // (every segment boundary inside a row tile adds a piece)
    return worst_passes <= num_sms / 2;
}

cudaError_t launch_gemm_sm100(const Arena& ar, const SlotSnapshot& snap, const CUtensorMap& tmap_B256,
                              const CUtensorMap& tmap_B128, const CUtensorMap& tmap_A, TmapCache* cache, const GemmArgs& a,
                              cudaStream_t stream)
{
    const bool dual = a.slot_ids2 != nullptr;
    if (dual && (a.G <= 0 || !a.y2)) return cudaErrorInvalidValue;
    const SplitChoice sc = gemm_pick_split(a.T, a.d_in, a.d_out, a.num_sms, a.split_bn, a.split_s);
    const int split = sc.split;
    const int bn = split ? sc.bn : gemm_pick_bn(a.T, a.d_out, a.num_sms);
    const int num_m = (a.T + kBM - 1) / kBM;
    const int num_n = (a.d_out + bn - 1) / bn;
    TmapCache local;   // (a call without a table-owned cache encodes its maps afresh)
    TmapCache* tc = cache ? cache : &local;
    CUtensorMap tx, tx0, tw, tu, ty, ty2;
    const CUtensorMap& tb = bn == 256 ? tmap_B256 : tmap_B128;
    const uint64_t u_set_rows = (uint64_t)(num_m + (a.G > 0 ? a.G : 1)) * kBM;
    const uint64_t u_rows = u_set_rows * (dual ? 3 : 1);
    const uint64_t xs = (uint64_t)a.d_in * 2, ys = (uint64_t)a.d_out * 2;
    if (!tc->get_2d(&tx, a.x, (uint64_t)a.d_in, (uint64_t)a.T, xs, kBK, kBM)) return cudaErrorInvalidValue;
    if (!tc->get_2d(&tx0, a.x_in_place ? a.x_in_place : a.x, (uint64_t)a.d_in, (uint64_t)a.T, xs, kBK, kBM)) return cudaErrorInvalidValue;
    if (!tc->get_2d(&tw, a.W0, (uint64_t)a.d_in, (uint64_t)a.d_out, xs, kBK, (uint32_t)bn)) return cudaErrorInvalidValue;
    if (!tc->get_2d(&tu, a.u_blocks, kRankPad, u_rows, kRankPad * 2, kBK, kBM)) return cudaErrorInvalidValue;
    if (!split) {   // (the split-K kernel stores its outputs with plain stores)
        if (!tc->get_2d(&ty, a.y, (uint64_t)a.d_out, (uint64_t)a.T, ys, kEpiChunkCols, 32)) return cudaErrorInvalidValue;
        if (!tc->get_2d(&ty2, dual ? a.y2 : a.y, (uint64_t)a.d_out, (uint64_t)a.T, ys, kEpiChunkCols, 32)) return cudaErrorInvalidValue;
    }
    GemmParams p;
    p.seg_offsets = a.seg_offsets; p.slot_ids = a.slot_ids; p.perm = a.perm; p.plan = a.plan;
    p.tile_identity = a.tile_identity;
    p.y = (__nv_bfloat16*)a.y; p.status = ar.status;
    p.slot_ids2 = a.slot_ids2; p.y2 = (__nv_bfloat16*)a.y2; p.u_set_rows = (int)u_set_rows;
    p.T = a.T; p.K = a.d_in; p.N = a.d_out; p.G = a.G; p.num_m = num_m; p.num_n = num_n;
    p.fused = (a.fused_shrink && !split && !dual) ? 1 : 0;
    p.tile_flags = ar.tile_flags; p.fuse_sync = ar.status + 4; p.u_out = const_cast<__nv_bfloat16*>(a.u_blocks);
    if (a.fused_shrink && !p.fused) return cudaErrorInvalidValue;   // (the caller asked gemm_can_fuse_shrink first)
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kGemmThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int nattr = 0;
    {   // with adapters the predecessor is the shrink kernel of this call, else the kernel waits at its top
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    if (split) {
        cfg.gridDim = dim3(split, num_n, num_m);
        cfg.dynamicSmemBytes = bn == 256 ? GemmCfg<256>::kSmemBytes : GemmCfg<128>::kSmemBytes;
        attr[nattr].id = cudaLaunchAttributeClusterDimension;
        attr[nattr].val.clusterDim.x = split;
        attr[nattr].val.clusterDim.y = 1;
        attr[nattr].val.clusterDim.z = 1;
        ++nattr;
        cfg.attrs = attr;
        cfg.numAttrs = nattr;
        if (bn == 256) return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_splitk_kernel<256>, tx, tx0, tw, tu, tb, snap, p);
        return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_splitk_kernel<128>, tx, tx0, tw, tu, tb, snap, p);
    }
    cfg.gridDim = dim3(min(num_m * num_n, a.num_sms));
    cfg.dynamicSmemBytes = bn == 256 ? GemmCfg<256>::kSmemBytes : GemmCfg<128>::kSmemBytes;
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    if (bn == 256) return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_kernel<256>, tx, tx0, tw, tu, tb, ty, ty2, tmap_A, snap, p);
    return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_kernel<128>, tx, tx0, tw, tu, tb, ty, ty2, tmap_A, snap, p);
}

}  // namespace lml
