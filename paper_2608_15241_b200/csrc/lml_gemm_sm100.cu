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
    static constexpr int kCtrlBytes = 256 + (kSegCache + 1) * 4 + 2 * kSegCache;   // barriers + segment cache (two slot arrays)
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
};

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1) lora_gemm_sm100_kernel(
    const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_x0,
    const __grid_constant__ CUtensorMap tmap_w,
    const __grid_constant__ CUtensorMap tmap_u, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_y2,
    const __grid_constant__ SlotSnapshot snap, const GemmParams p)
{
    using Cfg = GemmCfg<BN>;
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
    if (p.G == 0) {   // no shrink kernel ran before this one in the call: wait for foreign work here
        grid_dependency_wait();
        grid_launch_dependents();
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
                    grid_dependency_wait();
                    grid_launch_dependents();
                    lora = p.plan->lora_ok != 0;
                    lora_known = true;
                }
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

// kShrink: the same machinery computes the LoRA shrink.  A work item is a piece (block index b = tile m +
// segment g, see the shrink kernel): u = scale * x_tile . A_slot^T, a 128 x 64 product over all of K with
// the slot's 64 (zero-padded) rows of A in the place of W0; rows outside the segment are zeroed and the
// result is written as a bf16 u block.  Launched with a full dependency on the work before it.
template <int BN, bool kShrink = false>
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

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = (int)gridDim.x, rank = (int)blockIdx.x;   // the cluster spans the grid's x dimension
    const int n = (int)blockIdx.y;
    int m = (int)blockIdx.z;   // (shrink: the block index b; the tile follows from the lookup below)
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
        }
    }
    int piece_slot_id = -1, piece_lo = 0, piece_hi = 0;
    if (kShrink) {
        grid_launch_dependents();   // the GEMM behind this kernel may start on its base k-blocks
        const int b = (int)blockIdx.z;
        if (b == 0 && rank == 0) {   // one CTA validates the segment arrays for the whole call
            if (p.u_set_rows && threadIdx.x == 0) grid_dependency_wait();   // (a chained pass: see the launcher)
            int bad_off = 0, bad_slot = 0;
            for (int g = threadIdx.x; g < p.G; g += kGemmThreads) {
                const int s0 = __ldg(p.seg_offsets + g), s1 = __ldg(p.seg_offsets + g + 1);
                if (s1 < s0 || s0 < 0 || s1 > p.T) bad_off = 1;
                const int sl = __ldg(p.slot_ids + g);
                if (sl != -1 && s1 > s0 && slot_rank(snap, sl) == 0) bad_slot = 1;   // an empty segment may name anything
            }
            if (threadIdx.x == 0 && (__ldg(p.seg_offsets) != 0 || __ldg(p.seg_offsets + p.G) != p.T)) bad_off = 1;
            bad_off = __syncthreads_or(bad_off);
            bad_slot = __syncthreads_or(bad_slot);
            if (threadIdx.x == 0) {
                const_cast<PlanWord*>(p.plan)->lora_ok = bad_off ? 0 : 1;
                const unsigned f = (bad_off ? LML_FLAG_BAD_OFFSETS : 0u) | (bad_slot ? LML_FLAG_BAD_SLOT : 0u);
                if (f) atomicOr(p.status, f);
            }
        }
        __syncthreads();   // the segment cache is loaded
        if (threadIdx.x == 0) {   // which piece has block index b: the largest g with g + first tile of g <= b
            int lo = 0, hi = p.G;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                const int off = seg_cached ? seg_cache[mid] : __ldg(p.seg_offsets + mid);
                if (mid + off / kBM <= b) lo = mid; else hi = mid;
            }
            const int g = lo, mm = b - g;
            int found = 0, sl = -1, plo = 0, phi = 0;
            if (p.G > 0 && mm >= 0 && mm < p.num_m) {
                const int s0 = seg_cached ? seg_cache[g] : __ldg(p.seg_offsets + g);
                const int s1 = seg_cached ? seg_cache[g + 1] : __ldg(p.seg_offsets + g + 1);
                plo = max(max(s0, mm * kBM), 0);
                phi = min(min(s1, (mm + 1) * kBM), p.T);
                sl = __ldg(p.slot_ids + g);
                found = plo < phi && slot_rank(snap, sl) > 0;
            }
            ctrl->piece[0] = found; ctrl->piece[1] = sl; ctrl->piece[2] = plo; ctrl->piece[3] = phi;
        }
        __syncthreads();
        if (!ctrl->piece[0]) return;   // every CTA of the cluster shares b and leaves together; nothing reads this block
        piece_slot_id = ctrl->piece[1]; piece_lo = ctrl->piece[2]; piece_hi = ctrl->piece[3];
        m = piece_lo / kBM;
    }
    if (warp == 1) tmem_alloc(smem_u32(&ctrl->tmem_base), BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile int* abort = &ctrl->abort;
    if (!kShrink && p.G == 0) {   // no shrink kernel ran before this one in the call: wait for foreign work here
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
            auto piece_slot = [&](int g) -> int {
                int s0, s1, s;
                if (seg_cached) { s0 = seg_cache[g]; s1 = seg_cache[g + 1]; s = slot_cache[g]; }
                else {
                    s0 = __ldg(p.seg_offsets + g); s1 = __ldg(p.seg_offsets + g + 1); s = __ldg(p.slot_ids + g);
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
                ctrl->stage_info[stage] = 4u;
                mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                if (in_place) tma_load_2d(a_dst, &tmap_x0, bar, kb * kBK, row0);
                else tma_load_2d(a_dst, &tmap_x, bar, kb * kBK, row0);
                if (kShrink) tma_load_3d(a_dst + Cfg::kABytes, &tmap_b, bar, kb * kBK, 0, piece_slot_id);   // (tmap_b: the arena of A here)
                else tma_load_2d(a_dst + Cfg::kABytes, &tmap_w, bar, kb * kBK, n * BN);
                advance();
            }
            // this CTA's share of the tile's LoRA pieces
            bool lora = false;
            if (!kShrink && p.G > 0) {
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
                for (int g = g_first; g < g_end && ok; ++g) {
                    if (g % S != rank) continue;
                    const int s = piece_slot(g);
                    if (s < 0) continue;
                    ok = acquire();
                    if (!ok) break;
                    const uint32_t a_dst = tiles_addr + stage * Cfg::kStageBytes;
                    const uint32_t bar = smem_u32(&ctrl->full[stage]);
                    ctrl->stage_info[stage] = (uint32_t)((snap.rank[s] + 15) >> 4);
                    mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
                    tma_load_2d(a_dst, &tmap_u, bar, 0, (m + g) * kBM);
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
            uint32_t phase = 0, accumulate = 0;
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
#pragma unroll 4
                for (int k = 0; k < ksteps; ++k) {
                    umma_bf16(tmem_base, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, accumulate);
                    accumulate = 1;
                }
                umma_commit(smem_u32(&ctrl->empty[stage]));
                if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit(smem_u32(&ctrl->tmem_full[0]));
            ctrl->pad[0] = (int32_t)accumulate;   // 0: this CTA had no K at all, its accumulator holds nothing
        }
    }
    // ---------------------------------------------------------------------- exchange and reduction
    __syncwarp();   // (the producer's and the MMA issuer's other lanes waited here: the cluster barrier wants whole warps)
    bool ok = true;
    if (warp >= 2) {
        ok = mbar_wait_warp(smem_u32(&ctrl->tmem_full[0]), 0u, abort);   // this CTA's MMAs are complete: so are its loads
        tc_fence_after();
    }
    cluster_sync_all();   // every CTA of the cluster is done with its stage memory
    const int q = warp & 3;   // TMEM lane quarter an epilogue warp may read
    const int row = q * 32 + lane;
    if (warp >= 2 && ok) {
        const bool have = ctrl->pad[0] != 0;
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16);
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
            if (kShrink) {
                // the piece's u block: scale, zero outside the segment's rows, round; all 128 rows are written
                const bool mine = pos >= piece_lo && pos < piece_hi;
                const float sc = mine ? snap.scale[piece_slot_id] : 0.f;
                __nv_bfloat16* out = p.y + ((size_t)blockIdx.z * kBM + row) * kRankPad + col0;
                __nv_bfloat16* out_neg = p.y2 ? p.y2 + ((size_t)blockIdx.z * kBM + row) * kRankPad + col0 : nullptr;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 v;
                    v.x = pack_bf16(acc[8 * j + 0] * sc, acc[8 * j + 1] * sc);
                    v.y = pack_bf16(acc[8 * j + 2] * sc, acc[8 * j + 3] * sc);
                    v.z = pack_bf16(acc[8 * j + 4] * sc, acc[8 * j + 5] * sc);
                    v.w = pack_bf16(acc[8 * j + 6] * sc, acc[8 * j + 7] * sc);
                    if (!mine) v = make_uint4(0, 0, 0, 0);   // (0 * garbage may be a NaN)
                    *reinterpret_cast<uint4*>(out + j * 8) = v;
                    if (out_neg) *reinterpret_cast<uint4*>(out_neg + j * 8) = make_uint4(v.x ^ 0x80008000u, v.y ^ 0x80008000u, v.z ^ 0x80008000u, v.w ^ 0x80008000u);
                }
                continue;
            }
            if (!row_ok) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (col0 + j * 8 >= p.N) continue;
                uint4 v;
                v.x = pack_bf16(acc[8 * j + 0], acc[8 * j + 1]);
                v.y = pack_bf16(acc[8 * j + 2], acc[8 * j + 3]);
                v.z = pack_bf16(acc[8 * j + 4], acc[8 * j + 5]);
                v.w = pack_bf16(acc[8 * j + 6], acc[8 * j + 7]);
                *reinterpret_cast<uint4*>(p.y + (size_t)out_row * p.N + col0 + j * 8) = v;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.status, LML_FLAG_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, BN);
    }
}

// ---- CTA-pair variant ---------------------------------------------------------------------------------
// Two CTAs of a cluster share a 256 x 256 tile (cta_group::2).  CTA r of the pair owns rows
// [256 m2 + 128 r, +128): it stages its own 128 x 64 block of x and HALF of the W0 block (rows
// n0 + 128 r .. of W0), so a stage is 32 KB instead of 48 KB and the ring is six stages deep — the
// single-CTA kernel's four stages barely cover one TMA round trip.  The even CTA's MMA thread issues
// every MMA for both CTAs; the tensor cores fetch the other half of the W0 block from the peer's
// shared memory.  Barriers: full[] lives in the even CTA and counts both CTAs' TMA bytes; empty[] and
// tmem_full[] exist in both CTAs and are signalled by one commit addressed to both; tmem_empty[] lives
// in the even CTA and collects the epilogue warps of both.
// LoRA pieces: the pair walks the union of the segments that touch either half.  A CTA whose half
// does not meet a segment loads that stage's u operand from beyond the end of the u blocks, which
// TMA fills with zeros, so it adds nothing.
constexpr int kPairStages = 6;
constexpr int kPairBN = 256;
constexpr int kPairABytes = kBM * kBK * 2;                 // 16 KB: this CTA's rows of x (or of u)
constexpr int kPairBBytes = (kPairBN / 2) * kBK * 2;       // 16 KB: this CTA's half of the W0 (or B) block
constexpr int kPairStageBytes = kPairABytes + kPairBBytes;
constexpr int kPairEpiBytes = 4 * 2 * kEpiBufBytes;
constexpr int kPairCtrlBytes = 256 + (kSegCache + 1) * 4 + kSegCache;
constexpr int kPairSmemBytes = 1024 + kPairStages * kPairStageBytes + kPairEpiBytes + ((kPairCtrlBytes + 15) & ~15);

__global__ void __launch_bounds__(kGemmThreads, 1) lora_gemm_sm100_pair_kernel(
    const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
    const __grid_constant__ CUtensorMap tmap_u, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ SlotSnapshot snap,
    const GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t* tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    const uint32_t epi_addr = tiles_addr + kPairStages * kPairStageBytes;
    uint8_t* epi_ptr = tiles_ptr + kPairStages * kPairStageBytes;
    GemmCtrl* ctrl = reinterpret_cast<GemmCtrl*>(epi_ptr + kPairEpiBytes);
    int32_t* seg_cache = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(ctrl) + 256);
    int8_t* slot_cache = reinterpret_cast<int8_t*>(seg_cache + kSegCache + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = even CTA: issues the MMAs, owns full[] / tmem_empty[]
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_m2 = (p.num_m + 1) >> 1;             // 256-row tiles
    const int num_tiles = num_m2 * p.num_n;
    const int num_kb = (p.K + kBK - 1) / kBK;
    const bool seg_cached = p.G <= kSegCache;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctrl->tmem_full[a]), 1);
            mbar_init(smem_u32(&ctrl->tmem_empty[a]), 8);   // four epilogue warps in each CTA
        }
        ctrl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tmap(&tmap_x); prefetch_tmap(&tmap_w); prefetch_tmap(&tmap_u);
        prefetch_tmap(&tmap_b); prefetch_tmap(&tmap_y);
    }
    if (seg_cached && p.G > 0) {
        for (int g = threadIdx.x; g <= p.G; g += kGemmThreads) seg_cache[g] = __ldg(p.seg_offsets + g);
        for (int g = threadIdx.x; g < p.G; g += kGemmThreads) {
            int s = __ldg(p.slot_ids + g);
            slot_cache[g] = (int8_t)((s >= 0 && s < snap.max_slots && snap.rank[s] > 0) ? s : -1);
        }
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(&ctrl->tmem_base), 2 * kPairBN);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // both CTAs' barriers exist before either signals the other
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile int* abort = &ctrl->abort;
    if (p.G == 0) {   // no shrink kernel ran before this one in the call: wait for foreign work here
        grid_dependency_wait();
        grid_launch_dependents();
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            bool lora = false, lora_known = (p.G == 0);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            auto acquire = [&]() -> bool { return mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, abort); };
            auto advance = [&]() { if (++stage == kPairStages) { stage = 0; phase ^= 1u; } };
            const int u_rows_total = (p.num_m + (p.G > 0 ? p.G : 1)) * kBM;   // first row coordinate that TMA zero-fills
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                const int m2 = tile % num_m2, n = tile / num_m2;
                const int m = m2 * 2 + (int)rank;                      // this CTA's 128-row tile
                const int row0 = m * kBM, row1 = min(row0 + kBM, p.T);
                const int prow0 = m2 * 2 * kBM, prow1 = min(prow0 + 2 * kBM, p.T);   // the pair's rows
                int g_first = 0, g_end = 0, last_piece = -1;
                auto seg_at = [&](int g, int& s0, int& s1, int& s) {
                    if (seg_cached) { s0 = seg_cache[g]; s1 = seg_cache[g + 1]; s = slot_cache[g]; }
                    else {
                        s0 = __ldg(p.seg_offsets + g); s1 = __ldg(p.seg_offsets + g + 1); s = __ldg(p.slot_ids + g);
                        if (slot_rank(snap, s) == 0) s = -1;
                    }
                };
                // slot of the pair's piece for segment g (-1: none) and whether this CTA's half meets it
                auto pair_piece = [&](int g, bool& mine) -> int {
                    int s0, s1, s;
                    seg_at(g, s0, s1, s);
                    mine = min(s1, row1) > max(s0, row0);
                    if (min(s1, prow1) <= max(s0, prow0)) return -1;
                    return s;
                };
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    if (kb == num_kb - 1) {
                        if (!lora_known) {
                            grid_dependency_wait();   // plan word and u blocks come from the shrink kernel
                            grid_launch_dependents();
                            lora = p.plan->lora_ok != 0;
                            lora_known = true;
                        }
                        if (lora) {
                            if (seg_cached) {
                                int lo = 0, hi = p.G;
                                while (lo < hi) { int mid = (lo + hi) >> 1; if (seg_cache[mid + 1] > prow0) hi = mid; else lo = mid + 1; }
                                g_first = lo;
                                g_end = g_first;
                                while (g_end < p.G && seg_cache[g_end] < prow1) ++g_end;
                            } else {
                                g_first = seg_upper(p.seg_offsets, p.G, prow0);
                                g_end = g_first;
                                while (g_end < p.G && __ldg(p.seg_offsets + g_end) < prow1) ++g_end;
                            }
                            bool mine;
                            for (int g = g_first; g < g_end; ++g) if (pair_piece(g, mine) >= 0) last_piece = g;
                        }
                    }
                    ok = acquire();
                    if (!ok) break;
                    const uint32_t a_dst = tiles_addr + stage * kPairStageBytes;
                    const uint32_t bar = smem_u32(&ctrl->full[stage]);
                    if (rank == 0) {
                        ctrl->stage_info[stage] = 4u | ((kb == num_kb - 1 && last_piece < 0) ? 0x100u : 0u);
                        mbar_arrive_expect_tx(bar, 2 * kPairStageBytes);   // both CTAs' bytes land on this barrier
                    }
                    tma_load_2d_pair(a_dst, &tmap_x, bar, kb * kBK, row0);
                    tma_load_2d_pair(a_dst + kPairABytes, &tmap_w, bar, kb * kBK, n * kPairBN + (int)rank * (kPairBN / 2));
                    advance();
                }
                for (int g = g_first; g < g_end && ok; ++g) {
                    bool mine;
                    const int s = pair_piece(g, mine);
                    if (s < 0) continue;
                    ok = acquire();
                    if (!ok) break;
                    const uint32_t a_dst = tiles_addr + stage * kPairStageBytes;
                    const uint32_t bar = smem_u32(&ctrl->full[stage]);
                    if (rank == 0) {
                        const uint32_t ksteps = (uint32_t)((snap.rank[s] + 15) >> 4);
                        ctrl->stage_info[stage] = ksteps | (g == last_piece ? 0x100u : 0u);
                        mbar_arrive_expect_tx(bar, 2 * kPairStageBytes);
                    }
                    tma_load_2d_pair(a_dst, &tmap_u, bar, 0, mine ? (m + g) * kBM : u_rows_total);
                    tma_load_3d_pair(a_dst + kPairABytes, &tmap_b, bar, 0, n * kPairBN + (int)rank * (kPairBN / 2), s);
                    advance();
                }
            }
            for (int i = 0; i < kPairStages && ok; ++i) { ok = acquire(); advance(); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * kBM, kPairBN);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                ok = mbar_wait(smem_u32(&ctrl->tmem_empty[acc]), acc_phase ^ 1u, abort);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kPairBN);
                uint32_t accumulate = 0;
                bool more = true;
                for (int kb = 0; more; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->full[stage]), phase, abort);
                    if (!ok) break;
                    const uint32_t a_addr = tiles_addr + stage * kPairStageBytes;
                    const uint64_t adesc = umma_desc_k128(a_addr);
                    const uint64_t bdesc = umma_desc_k128(a_addr + kPairABytes);
                    int ksteps = 4;
                    if (kb >= num_kb - 1) {
                        const uint32_t info = ctrl->stage_info[stage];
                        ksteps = (int)(info & 0xffu);
                        more = (info & 0x100u) == 0;
                    }
#pragma unroll 4
                    for (int k = 0; k < ksteps; ++k) {
                        umma_bf16_pair(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit_pair(smem_u32(&ctrl->empty[stage]));   // frees the stage in both CTAs
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair(smem_u32(&ctrl->tmem_full[acc]));     // both CTAs' epilogues may read
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (both CTAs)
        const int q = warp & 3;
        const int ew = warp - 2;
        const uint32_t buf_addr0 = epi_addr + (uint32_t)(ew * 2 * kEpiBufBytes);
        uint8_t* buf_ptr0 = epi_ptr + ew * 2 * kEpiBufBytes;
        int acc = 0;
        uint32_t acc_phase = 0;
        int buf = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
            const int m2 = tile % num_m2, n = tile / num_m2;
            const int row_base = (m2 * 2 + (int)rank) * kBM + q * 32;
            ok = mbar_wait_warp(smem_u32(&ctrl->tmem_full[acc]), acc_phase, abort);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kPairBN);
#pragma unroll 1
            for (int c = 0; c < kPairBN / kEpiChunkCols; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(t_addr + (uint32_t)(c * kEpiChunkCols), r);
                tmem_ld_wait();
                if (c == kPairBN / kEpiChunkCols - 1) {
                    // accumulator fully read: tell the even CTA's MMA thread
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&ctrl->tmem_empty[acc]), 0));
                }
                const int col0 = n * kPairBN + c * kEpiChunkCols;
                if (col0 >= p.N || row_base >= p.T) continue;
                if (lane == 0) tma_store_wait_read<1>();
                __syncwarp();
                uint8_t* bp = buf_ptr0 + buf * kEpiBufBytes;
                const uint32_t ba = buf_addr0 + (uint32_t)(buf * kEpiBufBytes);
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
                if (p.perm == nullptr) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmap_y, ba, col0, row_base);
                        tma_store_commit();
                    }
                } else {
                    __syncwarp();
#pragma unroll
                    for (int pass = 0; pass < 4; ++pass) {
                        const int rr = pass * 8 + (lane >> 2), j = lane & 3;
                        const int pos = row_base + rr;
                        if (pos < p.T && col0 + j * 8 < p.N) {
                            const int row = __ldg(p.perm + pos);
                            if (row >= 0 && row < p.T) {
                                const int phys = j ^ ((rr >> 1) & 3);
                                uint4 v = *reinterpret_cast<const uint4*>(bp + rr * 64 + phys * 16);
                                *reinterpret_cast<uint4*>(p.y + (size_t)row * p.N + col0 + j * 8) = v;
                            }
                        }
                    }
                    __syncwarp();
                }
                buf ^= 1;
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all();
    }

    __syncthreads();
    cluster_sync_all();   // neither CTA leaves while the other may still read its tiles or signal its barriers
    if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.status, LML_FLAG_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 2 * kPairBN);
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
    e = cudaFuncSetAttribute(lora_gemm_sm100_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lora_gemm_sm100_splitk_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GemmCfg<256>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lora_gemm_sm100_splitk_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GemmCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lora_gemm_sm100_splitk_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GemmCfg<64>::kSmemBytes);
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
static SplitChoice gemm_pick_split(int T, int d_in, int d_out, int num_sms)
{
    static int max_clusters[2][kSplitMaxS + 1];
    static std::once_flag probed;
    if (const char* e = getenv("LML_GEMM_SPLIT")) {   // test knob: "<bn>x<split>", or 0 for no split
        int bn = 0, sp = 0;
        if (sscanf(e, "%dx%d", &bn, &sp) == 2 && (bn == 128 || bn == 256) && sp >= 2 && sp <= kSplitMaxS &&
            sp * ((bn / 32 + sp - 1) / sp) * 16384 <= GemmCfg<128>::kStages * GemmCfg<128>::kStageBytes)
            return {bn, sp};
        return {0, 0};
    }
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

// LML_FORCE_GEMM=pair|single overrides the choice below (a test knob: small problems would
// otherwise never reach the pair kernel).
static int gemm_forced_mode()
{
    static int mode = -1;
    if (mode < 0) {
        const char* e = getenv("LML_FORCE_GEMM");
        mode = !e ? 0 : (e[0] == 'p' ? 1 : (e[0] == 's' ? 2 : 0));
    }
    return mode;
}

bool gemm_pairs_forced() { return gemm_forced_mode() == 1; }

static bool gemm_use_pairs(int /*T*/, int /*d_out*/, int /*num_sms*/)
{
    // Measured on B200 (prefill_q_proj / mlp_up_gate, us per call): single-CTA tiles 66 / 314, CTA
    // pairs 74 / 349.  Pairs halve the W0 bytes each SM stages and give a six-stage ring, but the
    // cross-CTA barrier round trip costs more than that buys, so the single-CTA kernel is the
    // default and the pair kernel is selected only on request.
    return gemm_forced_mode() == 1;
}

cudaError_t launch_gemm_sm100(const Arena& ar, const SlotSnapshot& snap, const CUtensorMap& tmap_B,
                              const GemmArgs& a, cudaStream_t stream)
{
    const bool pairs = gemm_use_pairs(a.T, a.d_out, a.num_sms);
    const SplitChoice sc = (pairs || a.slot_ids2 != nullptr) ? SplitChoice{0, 0} : gemm_pick_split(a.T, a.d_in, a.d_out, a.num_sms);
    const int split = sc.split;
    const int bn = pairs ? kPairBN : (split ? sc.bn : gemm_pick_bn(a.T, a.d_out, a.num_sms));
    const int num_m = (a.T + kBM - 1) / kBM;
    const int num_n = (a.d_out + bn - 1) / bn;
    const uint32_t w_box_rows = pairs ? (uint32_t)(kPairBN / 2) : (uint32_t)bn;
    const bool dual = a.slot_ids2 != nullptr;
    if (dual && (pairs || a.G <= 0 || !a.y2)) return cudaErrorInvalidValue;
    CUtensorMap tx, tx0, tw, tu, ty, ty2, tb = tmap_B;
    if (!encode_tmap_2d(&tx, a.x, (uint64_t)a.d_in, (uint64_t)a.T, (uint64_t)a.d_in * 2, kBK, kBM)) return cudaErrorInvalidValue;
    if (!encode_tmap_2d(&tx0, a.x_in_place ? a.x_in_place : a.x, (uint64_t)a.d_in, (uint64_t)a.T, (uint64_t)a.d_in * 2, kBK, kBM)) return cudaErrorInvalidValue;
    if (!encode_tmap_2d(&tw, a.W0, (uint64_t)a.d_in, (uint64_t)a.d_out, (uint64_t)a.d_in * 2, kBK, w_box_rows)) return cudaErrorInvalidValue;
    const uint64_t u_set_rows = (uint64_t)(num_m + (a.G > 0 ? a.G : 1)) * kBM;
    const uint64_t u_rows = u_set_rows * (dual ? 3 : 1);
    if (!encode_tmap_2d(&tu, a.u_blocks, kRankPad, u_rows, kRankPad * 2, kBK, kBM)) return cudaErrorInvalidValue;
    if (!encode_tmap_2d(&ty, a.y, (uint64_t)a.d_out, (uint64_t)a.T, (uint64_t)a.d_out * 2, kEpiChunkCols, 32)) return cudaErrorInvalidValue;
    if (!encode_tmap_2d(&ty2, dual ? a.y2 : a.y, (uint64_t)a.d_out, (uint64_t)a.T, (uint64_t)a.d_out * 2, kEpiChunkCols, 32)) return cudaErrorInvalidValue;
    if (pairs || bn != 256) {
        if (!encode_tmap_3d(&tb, ar.B, kRankPad, (uint64_t)a.d_out, (uint64_t)snap.max_slots, kRankPad * 2,
                            (uint64_t)a.d_out * kRankPad * 2, kBK, w_box_rows, 1)) return cudaErrorInvalidValue;
    }
    GemmParams p;
    p.seg_offsets = a.seg_offsets; p.slot_ids = a.slot_ids; p.perm = a.perm; p.plan = a.plan;
    p.tile_identity = pairs ? nullptr : a.tile_identity;
    p.y = (__nv_bfloat16*)a.y; p.status = ar.status;
    p.slot_ids2 = a.slot_ids2; p.y2 = (__nv_bfloat16*)a.y2; p.u_set_rows = (int)u_set_rows;
    p.T = a.T; p.K = a.d_in; p.N = a.d_out; p.G = a.G; p.num_m = num_m; p.num_n = num_n;
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
    if (pairs) {
        const int pair_tiles = ((num_m + 1) / 2) * num_n;
        const int npairs = min(pair_tiles, a.num_sms / 2);
        cfg.gridDim = dim3(2 * npairs);
        cfg.dynamicSmemBytes = kPairSmemBytes;
        attr[nattr].id = cudaLaunchAttributeClusterDimension;
        attr[nattr].val.clusterDim.x = 2;
        attr[nattr].val.clusterDim.y = 1;
        attr[nattr].val.clusterDim.z = 1;
        ++nattr;
        cfg.attrs = attr;
        cfg.numAttrs = nattr;
        return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_pair_kernel, tx, tw, tu, tb, ty, snap, p);
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
    if (bn == 256) return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_kernel<256>, tx, tx0, tw, tu, tb, ty, ty2, snap, p);
    return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_kernel<128>, tx, tx0, tw, tu, tb, ty, ty2, snap, p);
}


// The LoRA shrink on the tensor cores: the shrink form of the split-K kernel, one cluster per block index.
// Returns cudaErrorNotSupported when the caller should use the mma.sync kernel instead.
cudaError_t launch_shrink_sm100(const Arena& ar, const SlotSnapshot& snap, const void* x, int T, int d_in,
                                const int32_t* seg_offsets, const int32_t* slot_ids, int G, const void* x_in_place,
                                const int32_t* tile_identity, PlanWord* plan, __nv_bfloat16* u_blocks,
                                cudaStream_t stream, bool chained, __nv_bfloat16* u_blocks_neg)
{
    static int max_clusters[kSplitMaxS + 1];
    static int num_sms = 0;
    static std::once_flag probed;
    std::call_once(probed, [&]() {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return;
        }
        for (int S = 1; S <= kSplitMaxS; ++S) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(S, 1, sms / S);
            cfg.blockDim = dim3(kGemmThreads);
            cfg.dynamicSmemBytes = GemmCfg<64>::kSmemBytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, lora_gemm_sm100_splitk_kernel<64, true>, &cfg) != cudaSuccess) { n = 0; (void)cudaGetLastError(); }
            max_clusters[S] = n;
        }
        num_sms = sms;
    });
    if (num_sms == 0) return cudaErrorNotSupported;
    const int num_m = (T + kBM - 1) / kBM, num_kb = (d_in + kBK - 1) / kBK;
    const int blocks = num_m + (G > 0 ? G : 1);
    // as many CTAs per piece as still leaves every block index a cluster that is resident at once
    int split = 1;
    for (int S = 2; S <= kSplitMaxS; ++S)
        if (blocks <= max_clusters[S] && num_kb >= 2 * S) split = S;
    CUtensorMap tx, tx0, ta;
    if (!encode_tmap_2d(&tx, x, (uint64_t)d_in, (uint64_t)T, (uint64_t)d_in * 2, kBK, kBM)) return cudaErrorInvalidValue;
    if (!encode_tmap_2d(&tx0, x_in_place ? x_in_place : x, (uint64_t)d_in, (uint64_t)T, (uint64_t)d_in * 2, kBK, kBM)) return cudaErrorInvalidValue;
    if (!encode_tmap_3d(&ta, ar.A, (uint64_t)d_in, kRankPad, (uint64_t)snap.max_slots, (uint64_t)d_in * 2,
                        (uint64_t)d_in * kRankPad * 2, kBK, kRankPad, 1)) return cudaErrorInvalidValue;
    GemmParams p = {};
    p.seg_offsets = seg_offsets; p.slot_ids = slot_ids; p.perm = nullptr; p.plan = plan;
    p.tile_identity = tile_identity;
    p.y = u_blocks; p.y2 = u_blocks_neg; p.status = ar.status; p.slot_ids2 = nullptr;
    p.u_set_rows = chained ? 1 : 0;
    p.T = T; p.K = d_in; p.N = kRankPad; p.G = G; p.num_m = num_m; p.num_n = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(split, 1, blocks);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = GemmCfg<64>::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = split; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // only a chained pass starts before its predecessor ends
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, lora_gemm_sm100_splitk_kernel<64, true>, tx, tx0, tx, tx, ta, snap, p);
}

}  // namespace lml
