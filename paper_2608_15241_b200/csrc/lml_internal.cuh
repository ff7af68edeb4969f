// Internal declarations shared by the sm_100a kernels and the host API of the mixed-adapter
// LoRA linear library.  Not part of the public ABI.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "lora_mixed_linear.h"

namespace lml {

constexpr int kMaxSlots = LML_MAX_SLOTS;
constexpr int kRankPad = 64;          // adapters are stored zero-padded to this rank
constexpr int kRankCompact = 16;      // ... and B a second time, padded to this rank only, where the rank allows
constexpr int kTileM = 128;           // token rows per GEMM tile and per shrink piece block
constexpr int kDecodeMaxT = LML_DECODE_MAX_TOKENS;
constexpr int kMaxAdapterIds = LML_MAX_ADAPTER_IDS;
constexpr int kFuseMaxTiles = 4096;   // row tiles of a call whose shrink can run inside the GEMM kernel (524288 tokens)   // adapter ids that can be resolved on the device

// Per-call snapshot of the slot table, passed by value as a kernel parameter so that a later
// register / retire cannot change a call that is already enqueued.
struct SlotSnapshot {
    uint8_t rank[kMaxSlots];   // 0 = slot not live.  First, with max_slots right behind: what a kernel needs
    int32_t max_slots;         // first sits in one or two lines of the parameter cache (a miss there costs
    float scale[kMaxSlots];    // as much as a trip to L2)
    uint16_t gen[kMaxSlots];   // registration counter of the entry in the slot: what a word of the adapter map must name
};

// Device-resident pieces of a table.
struct Arena {
    __nv_bfloat16* A;   // [max_slots][kRankPad][d_in]   rows >= rank are zero
    __nv_bfloat16* B;   // [max_slots][d_out][kRankPad]  columns >= rank are zero
    __nv_bfloat16* Bc;  // [max_slots][d_out][kRankCompact]: the same rows, 32 bytes each, for slots of rank <= kRankCompact
                        // (what the decode kernel reads: it needs a row's real columns only, a quarter of the padded row)
    uint32_t* status;   // sticky LML_FLAG_* bits
    int32_t* tile_flags;    // [kFuseMaxTiles] fused shrink of the prefill GEMM: row tile m's u blocks are written (= epoch + 1; the epoch is word 4 of status)
    int32_t* adapter_map;   // [kMaxAdapterIds] serving entry of each adapter id: slot | generation << 8, -1 = none; written by lml_publish
    unsigned long long* dec_u;   // [kDecMaxBlocks][kDecExchStride] the decode kernel's exchange blocks, one per part of a launch that works on this table
};

inline int32_t adapter_map_word(int slot, uint16_t gen) { return (int32_t)((uint32_t)slot | ((uint32_t)gen << 8)); }

// Workspace header written by the shrink kernels and read by the kernels that follow.
struct PlanWord {
    int32_t lora_ok;    // 1 = seg_offsets well formed, expand steps may run
    int32_t pad[63];
};

// ---- kernel launchers (each enqueues on `stream` and returns the launch error) ------------

cudaError_t launch_pack_adapter(const Arena& ar, int slot, const void* A, const void* B, int rank,
                                int d_in, int d_out, cudaStream_t stream);

cudaError_t launch_set_word(int32_t* dst, int32_t value, cudaStream_t stream);
cudaError_t launch_clear_word_if(int32_t* dst, int32_t expected, cudaStream_t stream);   // *dst = -1 if it still holds `expected`
cudaError_t aux_init();   // sets the dynamic shared memory attribute of the gradient kernel
// per-chunk segment arrays ([offsets (G + 1) | slot ids (G)] every `stride` ints) of a call done in chunks of `rows` rows
cudaError_t launch_clip_segments(const int32_t* seg_offsets, const int32_t* slot_ids, int G, int T, int rows, int chunks,
                                 int32_t* out, int stride, cudaStream_t stream);
// inputs of a decode call out of pinned host memory (device-accessible pointers) into device staging; x_bytes a multiple of 16
cudaError_t launch_stage_host_inputs(const void* x_host, void* x_dev, size_t x_bytes, const int32_t* so_host, int32_t* so_dev,
                                     int n_so, const int32_t* ids_host, int32_t* ids_dev, int n_ids,
                                     const int32_t* perm_host, int32_t* perm_dev, int n_perm, cudaStream_t stream);
// (A', B') = (B^T, A^T) of a forward adapter A [rank][K], B [N][rank] into slot `slot` of the transposed table's arena
cudaError_t launch_pack_adapter_transposed(const Arena& arT, int slot, const void* A, const void* B, int rank,
                                           int K, int N, cudaStream_t stream);
// out_s += P_s^T . Q_s per slot (adapter gradients); mode 0: out[slot][j][c], mode 1: out[slot][c][j]
cudaError_t launch_weight_grad(const SlotSnapshot& snap, const __nv_bfloat16* pieces, const void* Q, int T, int C,
                               const int32_t* seg_offsets, const int32_t* slot_ids, int G, float* out, int mode,
                               cudaStream_t stream,   // optionally a second gradient in the same launch:
                               const __nv_bfloat16* pieces2 = nullptr, const void* Q2 = nullptr, int C2 = 0,
                               float* out2 = nullptr, int mode2 = 0);
cudaError_t launch_segment_tokens(const Arena& ar, const SlotSnapshot& snap, const int32_t* token_slots,
                                  int T, int32_t* perm, int32_t* seg_offsets, int32_t* seg_slot_ids,
                                  cudaStream_t stream, bool by_adapter = false);   // by_adapter: the ids are adapter ids, resolved through ar.adapter_map

// u blocks: block b = (tile m) + (segment g) holds the 128 x 64 bf16 values scale*(x.A^T) of
// the rows of tile m that belong to segment g, zero elsewhere.
// x_in_place / tile_identity: rows of tiles marked identity are read from x_in_place instead of x.
cudaError_t launch_shrink_pieces(const Arena& ar, const SlotSnapshot& snap, const void* x, int T,
                                 int d_in, const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                                 const void* x_in_place, const int32_t* tile_identity, PlanWord* plan,
                                 __nv_bfloat16* u_blocks, cudaStream_t stream, int chained = 0,   // 1: a further pass of the same call, may run beside the one before; 2: behind the call's row-gather kernel
                                 __nv_bfloat16* u_blocks_neg = nullptr);                              // optional second copy of the blocks, negated

// tile_identity[m] = 1: tile m's perm is the identity, its rows were not copied and stay in place.
// token-form calls of one row tile: binding and shrink in one launch, tokens in their order (see the kernel)
cudaError_t launch_bind_shrink_tile(const Arena& ar, const SlotSnapshot& snap, const int32_t* token_slots, int T, int d_in,
                                    const void* x, int32_t* seg_offsets, int32_t* seg_slot_ids, int G, PlanWord* plan,
                                    void* u_blocks, int threads, cudaStream_t stream, bool by_adapter);
cudaError_t launch_gather_rows(const void* x, const int32_t* perm, int T, int d_in, void* x_grouped,
                               int32_t* tile_identity, bool allow_skip, uint32_t* status, cudaStream_t stream);

struct GemmArgs {
    const void* x;            // rows in position order (already gathered when perm is used)
    const void* x_in_place;   // perm form: the caller's x, read for tiles whose perm is the identity
    const int32_t* tile_identity;   // perm form: 1 per 128-row tile that was left in place, else NULL
    const void* W0;
    void* y;
    const int32_t* perm;      // NULL or position -> output row
    const int32_t* seg_offsets;
    const int32_t* slot_ids;
    const PlanWord* plan;
    const __nv_bfloat16* u_blocks;
    const int32_t* slot_ids2 = nullptr;   // dual form: second slot per segment; u_blocks then holds three sets of
    void* y2 = nullptr;                   // (num_m + G) blocks: first slots, second slots, first slots negated
    int T, d_in, d_out, G;
    int num_sms;
    bool fused_shrink = false;         // no shrink kernel ran: the GEMM kernel computes the u blocks itself (see gemm_can_fuse_shrink)
    int split_bn = -1, split_s = -1;   // the table's split-K override: -1 = the library chooses, 0 = off, else the forced shape
    bool overlap_with_previous;   // launch as a programmatic dependent of the shrink kernel before it
};
// Tensor maps of caller buffers, kept per table and found again by (pointer, shape, box).
struct TmapCache {
    static constexpr int kEntries = 32;
    struct Key { const void* base; uint64_t inner, outer, stride; uint32_t box_inner, box_outer; };
    Key keys[kEntries];
    CUtensorMap maps[kEntries];
    int used = 0, next = 0;
    std::mutex mu;
    bool get_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint64_t stride_bytes,
                uint32_t box_inner, uint32_t box_outer);
};
bool gemm_split_override(int* bn_out, int* split_out);
// tmap_B256 / tmap_B128: the table's maps of its packed B arena for 256- and 128-column tiles.
// Returns cudaErrorInvalidValue if a tensor map cannot be encoded.
bool gemm_can_fuse_shrink(int T, int d_in, int d_out, int G, int num_sms, int split_bn, int split_s);
// tmap_A: the table's map of its packed A arena ([max_slots][64][d_in], box 64 x 64 x 1), for the fused shrink.
cudaError_t launch_gemm_sm100(const Arena& ar, const SlotSnapshot& snap, const CUtensorMap& tmap_B256,
                              const CUtensorMap& tmap_B128, const CUtensorMap& tmap_A, TmapCache* cache, const GemmArgs& a,
                              cudaStream_t stream);
cudaError_t gemm_sm100_init(int device);
cudaError_t shrink_init();   // both set the dynamic shared memory attributes of their kernels
bool encode_tmap_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer,
                    uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer);
bool encode_tmap_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1,
                    uint32_t b2);

// The decode kernel's exchange block, through which the CTAs of a launch hand one another u = scale * x.A^T: 16 x kRankPad
// entries (an fp32 value beside the mark of the launch that wrote it, one 64-bit word), then three 32-bit words: the mark
// of the last launch that finished on this block, the CTAs that have left, the entries written.  All zero to begin with.
constexpr int kDecExchEntries = 16 * kRankPad;
constexpr int kDecExchStride = kDecExchEntries + 8;   // 64-bit words per block
constexpr int kDecMaxBlocks = 8;   // parts of one decode launch at most (projections, bindings, blocks of 16 tokens)
struct DecodeArgs {
    const void* x;
    const void* W0;
    void* y;
    const int32_t* perm;
    const int32_t* seg_offsets;
    const int32_t* slot_ids;
    const int32_t* token_slots = nullptr;   // instead of segments: one slot id per row of x (then G is 1 and perm is null)
    bool by_adapter = false;                // the ids in token_slots are adapter ids, resolved through the table's device map
    unsigned long long* exch = nullptr;   // exchange block of the call (kDecExchStride words); null: the table's own, by order of use in the launch
    int T, d_in, d_out, G;
    int num_sms;
};
cudaError_t decode_init();   // sets the dynamic shared memory attributes
int decode_patience();       // LML_DECODE_PATIENCE or the default, in clock cycles
cudaError_t launch_decode(const Arena& ar, const SlotSnapshot& snap, const DecodeArgs& a,
                          cudaStream_t stream, int* launches);
// P <= kDecMaxBlocks parts in one launch (d_in and num_sms equal for all; at most LML_MAX_PROJECTIONS distinct tables):
// projections that read the same x, the two bindings of a dual call, blocks of 16 tokens of a larger batch.
cudaError_t launch_decode_multi(const Arena* const* ars, const SlotSnapshot* snaps, const DecodeArgs* args, int P,
                                cudaStream_t stream);

// Every kernel of the library is launched as a programmatic dependent of whatever precedes it on
// the stream and executes griddepcontrol.wait before it touches global memory (unless its
// predecessor is the library's own kernel of the same call, which has already waited).  The wait
// costs nothing when the predecessor does not trigger early, and otherwise hides launch latency and
// the prologue behind the predecessor's tail.
inline void pdl_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream)
{
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

// ---- small device helpers -------------------------------------------------------------------

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&p);
}

__device__ __forceinline__ uint4 ldg_nc_v4(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Segment lookup shared by the kernels.  seg_offsets is assumed monotone (the shrink kernel
// validates it and clears PlanWord::lora_ok otherwise); all results are clamped so that a
// malformed array can only produce wrong-but-in-range indices.
//
// first segment whose end lies beyond `pos`
__device__ __forceinline__ int seg_upper(const int32_t* __restrict__ seg_offsets, int G, int pos)
{
    int lo = 0, hi = G;   // answer in [0, G]
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (__ldg(seg_offsets + mid + 1) > pos) hi = mid; else lo = mid + 1;
    }
    return lo;
}

__device__ __forceinline__ int slot_rank(const SlotSnapshot& snap, int slot)
{
    return (slot >= 0 && slot < snap.max_slots) ? (int)snap.rank[slot] : 0;
}

// adapter id -> serving slot through the table's device map.  -1 stays -1 (no adapter); an id out of range,
// without a serving version, or whose map word names an entry that is no longer the one in that slot
// (retired, slot taken by another registration since) gives -2: no adapter, and the caller raises the flag.
__device__ __forceinline__ int resolve_adapter(const SlotSnapshot& snap, const int32_t* __restrict__ adapter_map, int id)
{
    if (id == -1) return -1;
    if (id < 0 || id >= kMaxAdapterIds) return -2;
    const int v = __ldg(adapter_map + id);
    if (v < 0) return -2;
    const int slot = v & 0xff;
    if (slot >= snap.max_slots || snap.rank[slot] == 0 || snap.gen[slot] != (uint16_t)((uint32_t)v >> 8)) return -2;
    return slot;
}

}  // namespace lml
