// Host side of the C ABI: the adapter slot table, argument validation, workspace layout and
// dispatch to the decode / prefill kernels.  See include/lora_mixed_linear.h for the contract.
#include <cstdlib>
#include <new>

#include "lml_table.cuh"

using namespace lml;

namespace {

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Workspace layout of the prefill path: [PlanWord][tile_identity][u blocks][gathered x (perm form only)];
// the decode path uses [PlanWord][..][u fp32 16x64].
struct WsLayout {
    size_t plan_off, ident_off, u_off, xg_off, total;
};
WsLayout ws_layout(const lml_table* t, int T, int G, int u_sets = 1)
{
    WsLayout w;
    w.plan_off = 0;
    const size_t num_m = (size_t)(T + kTileM - 1) / kTileM;
    w.ident_off = round_up(sizeof(PlanWord), 256);
    w.u_off = round_up(w.ident_off + (num_m + 1) * sizeof(int32_t), 1024);
    size_t u_bytes = (size_t)u_sets * (num_m + (size_t)(G > 0 ? G : 1)) * kTileM * kRankPad * sizeof(__nv_bfloat16);
    w.xg_off = w.u_off + round_up(u_bytes, 1024);
    w.total = w.xg_off + round_up((size_t)T * t->d_in * sizeof(__nv_bfloat16), 1024);
    return w;
}

}  // namespace

static void free_table_resources(lml_table* t)
{
    cudaFree(t->arena.A); cudaFree(t->arena.B); cudaFree(t->arena.Bc); cudaFree(t->arena.status); cudaFree(t->arena.adapter_map); cudaFree(t->arena.tile_flags); cudaFree(t->arena.dec_u);
    if (t->copy_in) cudaStreamDestroy(t->copy_in);
    if (t->copy_out) cudaStreamDestroy(t->copy_out);
    if (t->ev_begin) cudaEventDestroy(t->ev_begin);
    if (t->ev_done) cudaEventDestroy(t->ev_done);
    if (t->ev_map) cudaEventDestroy(t->ev_map);
    for (int c = 0; c < lml_table::kHostChunks; ++c) {
        if (t->ev_in[c]) cudaEventDestroy(t->ev_in[c]);
        if (t->ev_layer[c]) cudaEventDestroy(t->ev_layer[c]);
    }
    (void)cudaGetLastError();
}

extern "C" {

const char* lml_status_string(lml_status s)
{
    switch (s) {
        case LML_OK: return "ok";
        case LML_ERR_INVALID_ARG: return "invalid argument";
        case LML_ERR_BAD_SLOT: return "bad slot";
        case LML_ERR_TABLE_FULL: return "slot table full";
        case LML_ERR_DUPLICATE: return "adapter version already resident";
        case LML_ERR_NOT_FOUND: return "adapter version not resident";
        case LML_ERR_UNSUPPORTED: return "device is not sm_100";
        case LML_ERR_CUDA: return "CUDA call failed";
        case LML_ERR_TIMEOUT: return "device wait timed out";
        case LML_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case LML_ERR_TOO_LARGE: return "call exceeds the fixed capacity of this entry point";
    }
    return "unknown status";
}

lml_status lml_table_create(lml_table** out, int device, int d_in, int d_out, int max_slots)
{
    if (!out) return LML_ERR_INVALID_ARG;
    *out = nullptr;
    if (device < 0 || d_in <= 0 || d_out <= 0 || (d_in % 8) || (d_out % 8) || max_slots < 1 ||
        max_slots > kMaxSlots)
        return LML_ERR_INVALID_ARG;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
    if (device >= count) return LML_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
    if (prop.major != 10) return LML_ERR_UNSUPPORTED;
    DeviceGuard guard(device);
    if (!guard.ok) return LML_ERR_CUDA;

    lml_table* t = new (std::nothrow) lml_table();
    if (!t) return LML_ERR_CUDA;
    t->device = device; t->d_in = d_in; t->d_out = d_out; t->max_slots = max_slots;
    t->num_sms = prop.multiProcessorCount;
    const size_t a_bytes = (size_t)max_slots * kRankPad * d_in * sizeof(__nv_bfloat16);
    const size_t b_bytes = (size_t)max_slots * d_out * kRankPad * sizeof(__nv_bfloat16);
    bool ok = cudaMalloc(&t->arena.A, a_bytes) == cudaSuccess;
    ok = ok && cudaMalloc(&t->arena.B, b_bytes) == cudaSuccess;
    const size_t bc_bytes = (size_t)max_slots * d_out * kRankCompact * sizeof(__nv_bfloat16);
    ok = ok && cudaMalloc(&t->arena.Bc, bc_bytes) == cudaSuccess;
    ok = ok && cudaMemset(t->arena.Bc, 0, bc_bytes) == cudaSuccess;
    ok = ok && cudaMalloc(&t->arena.status, 256) == cudaSuccess;
    ok = ok && cudaMalloc(&t->arena.adapter_map, kMaxAdapterIds * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemset(t->arena.A, 0, a_bytes) == cudaSuccess;
    ok = ok && cudaMemset(t->arena.B, 0, b_bytes) == cudaSuccess;
    ok = ok && cudaMemset(t->arena.status, 0, 256) == cudaSuccess;
    const size_t dec_u_bytes = (size_t)kDecMaxBlocks * kDecExchStride * sizeof(unsigned long long);
    ok = ok && cudaMalloc(&t->arena.dec_u, dec_u_bytes) == cudaSuccess;
    ok = ok && cudaMemset(t->arena.dec_u, 0, dec_u_bytes) == cudaSuccess;   // mark 0: written by no launch
    ok = ok && cudaMemset(t->arena.adapter_map, 0xff, kMaxAdapterIds * sizeof(int32_t)) == cudaSuccess;   // -1: no serving version
    ok = ok && cudaMalloc(&t->arena.tile_flags, kFuseMaxTiles * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemset(t->arena.tile_flags, 0, kFuseMaxTiles * sizeof(int32_t)) == cudaSuccess;
    ok = ok && gemm_sm100_init(device) == cudaSuccess;
    ok = ok && shrink_init() == cudaSuccess;
    ok = ok && decode_init() == cudaSuccess;
    ok = ok && aux_init() == cudaSuccess;
    ok = ok && encode_tmap_3d(&t->tmap_B256, t->arena.B, kRankPad, (uint64_t)d_out, (uint64_t)max_slots,
                              kRankPad * 2, (uint64_t)d_out * kRankPad * 2, 64, 256, 1);
    ok = ok && encode_tmap_3d(&t->tmap_B128, t->arena.B, kRankPad, (uint64_t)d_out, (uint64_t)max_slots,
                              kRankPad * 2, (uint64_t)d_out * kRankPad * 2, 64, 128, 1);
    ok = ok && encode_tmap_3d(&t->tmap_A, t->arena.A, (uint64_t)d_in, kRankPad, (uint64_t)max_slots, (uint64_t)d_in * 2,
                              (uint64_t)d_in * kRankPad * 2, 64, 64, 1);
    gemm_split_override(&t->split_bn, &t->split_s);   // the test knobs are read here, never on the hot path
    if (const char* e = getenv("LML_FUSE_SHRINK")) t->fuse_shrink = e[0] != '0';
    // (two row tiles where the rows of x are short enough for the GEMM's CTAs to get resident beside the binding kernel's:
    // 256 tokens 29 / 45 us against 34 / 50 on the grouped path on 4096 x 4096 / 11008 x 4096; from 512 tokens on, and on
    // 4096 x 11008 from 256 on, a piece per slot and tile costs the GEMM more than grouping the rows)
    t->one_tile_tokens = d_in <= 4096 ? 2 * kTileM : kTileM;
    if (const char* e = getenv("LML_ONE_TILE")) t->one_tile_tokens = e[0] != '0' ? t->one_tile_tokens : 0;
    if (const char* e = getenv("LML_ONE_TILE_TOKENS")) t->one_tile_tokens = atoi(e) < 0 ? 0 : (atoi(e) > 8 * kTileM ? 8 * kTileM : atoi(e));
    if (const char* e = getenv("LML_BIND_THREADS")) t->bind_threads = atoi(e);
    if (const char* e = getenv("LML_DECODE_BLOCK_TOKENS")) t->dec_block_tokens = atoi(e) < 0 ? 0 : (atoi(e) > kDecMaxBlocks * kDecodeMaxT ? kDecMaxBlocks * kDecodeMaxT : atoi(e));
    ok = ok && cudaEventCreateWithFlags(&t->ev_map, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&t->copy_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&t->copy_out, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&t->ev_begin, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&t->ev_done, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; c < lml_table::kHostChunks; ++c) {
        ok = ok && cudaEventCreateWithFlags(&t->ev_in[c], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&t->ev_layer[c], cudaEventDisableTiming) == cudaSuccess;
    }
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_table_resources(t);
        delete t;
        return LML_ERR_CUDA;
    }
    *out = t;
    return LML_OK;
}

lml_status lml_table_destroy(lml_table* t)
{
    if (!t) return LML_ERR_INVALID_ARG;
    {
        DeviceGuard guard(t->device);
        free_table_resources(t);
    }
    delete t;
    return LML_OK;
}

lml_status register_adapter(lml_table* t, int adapter_id, int version, const void* A, const void* B, int rank,
                            float scale, void* stream, int* slot_out)
{
    if (!t || !A || !B || !slot_out || rank < 1 || rank > LML_MAX_RANK || !aligned16(A) || !aligned16(B) ||
        !(scale == scale))
        return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    int free_slot = -1;
    for (int i = 0; i < t->max_slots; ++i) {
        const auto& e = t->entries[i];
        if (e.live && e.adapter_id == adapter_id && e.version == version) return LML_ERR_DUPLICATE;
        if (!e.live && free_slot < 0) free_slot = i;
    }
    if (free_slot < 0) return LML_ERR_TABLE_FULL;
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    // a slot that a retire freed is overwritten only behind the kernel that took it out of the device map
    if (t->map_clear_recorded && cudaStreamWaitEvent((cudaStream_t)stream, t->ev_map, 0) != cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    if (launch_pack_adapter(t->arena, free_slot, A, B, rank, t->d_in, t->d_out, (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    auto& e = t->entries[free_slot];
    e.adapter_id = adapter_id; e.version = version; e.rank = rank; e.scale = scale;
    e.state = LML_STATE_RESIDENT; e.pins = 0;
    e.gen = ++t->next_gen;
    e.live = true;   // published last: the entry is complete before it becomes visible
    *slot_out = free_slot;
    return LML_OK;
}

lml_status register_adapter_transposed(lml_table* t_T, int adapter_id, int version, const void* A, const void* B, int rank,
                                       float scale, void* stream, int* slot_out)
{
    // A [rank][K], B [N][rank] are the FORWARD layer's matrices; t_T has d_in = N and d_out = K
    if (!t_T || !A || !B || !slot_out || rank < 1 || rank > LML_MAX_RANK || !aligned16(A) || !aligned16(B) || !(scale == scale))
        return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t_T->mu);
    int free_slot = -1;
    for (int i = 0; i < t_T->max_slots; ++i) {
        const auto& e = t_T->entries[i];
        if (e.live && e.adapter_id == adapter_id && e.version == version) return LML_ERR_DUPLICATE;
        if (!e.live && free_slot < 0) free_slot = i;
    }
    if (free_slot < 0) return LML_ERR_TABLE_FULL;
    DeviceGuard guard(t_T->device);
    if (!guard.ok) return LML_ERR_CUDA;
    if (t_T->map_clear_recorded && cudaStreamWaitEvent((cudaStream_t)stream, t_T->ev_map, 0) != cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    if (launch_pack_adapter_transposed(t_T->arena, free_slot, A, B, rank, /*K=*/t_T->d_out, /*N=*/t_T->d_in,
                                       (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    auto& e = t_T->entries[free_slot];
    e.adapter_id = adapter_id; e.version = version; e.rank = rank; e.scale = scale;
    e.state = LML_STATE_RESIDENT; e.pins = 0;
    e.gen = ++t_T->next_gen;
    e.live = true;
    *slot_out = free_slot;
    return LML_OK;
}

lml_status retire_version_on(lml_table* t, int adapter_id, int version, void* stream)
{
    if (!t) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    for (int i = 0; i < t->max_slots; ++i) {
        auto& e = t->entries[i];
        if (e.live && e.adapter_id == adapter_id && e.version == version) {
            if (e.state == LML_STATE_SERVING) {
                // No longer the adapter's serving version: calls that name the adapter must stop resolving to it.
                // The word is cleared in stream order, like the publish that set it, and only if it still names
                // this entry (a newer publish of the adapter stays).  The event lets later registrations order
                // themselves behind the clear before they reuse the slot.
                DeviceGuard guard(t->device);
                bool ok = guard.ok;
                ok = ok && launch_clear_word_if(t->arena.adapter_map + adapter_id, adapter_map_word(i, e.gen), (cudaStream_t)stream) == cudaSuccess;
                ok = ok && cudaEventRecord(t->ev_map, (cudaStream_t)stream) == cudaSuccess;
                if (!ok) {
                    cudaGetLastError();
                    return LML_ERR_CUDA;
                }
                t->map_clear_recorded = true;
            }
            if (e.pins > 0) e.state = LML_STATE_RETIRING;   // freed by the last unpin
            else e.live = false;
            return LML_OK;
        }
    }
    return LML_ERR_NOT_FOUND;
}

lml_status retire_version(lml_table* t, int adapter_id, int version)
{
    return retire_version_on(t, adapter_id, version, nullptr);   // the legacy default stream
}

lml_status lml_publish(lml_table* t, int adapter_id, int version, void* stream, int* previous_version_out)
{
    if (!t || adapter_id < 0 || adapter_id >= kMaxAdapterIds) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    int slot = -1, prev = -1;
    for (int i = 0; i < t->max_slots; ++i) {
        const auto& e = t->entries[i];
        if (!e.live || e.adapter_id != adapter_id) continue;
        if (e.version == version && e.state != LML_STATE_RETIRING) slot = i;
        else if (e.state == LML_STATE_SERVING) prev = i;
    }
    if (slot < 0) return LML_ERR_NOT_FOUND;
    if (previous_version_out) *previous_version_out = prev >= 0 ? t->entries[prev].version : -1;
    if (t->entries[slot].state == LML_STATE_SERVING) return LML_OK;   // already the serving version
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    // the controlled publication point: one 4-byte store, in stream order
    if (launch_set_word(t->arena.adapter_map + adapter_id, adapter_map_word(slot, t->entries[slot].gen), (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    t->entries[slot].state = LML_STATE_SERVING;
    if (prev >= 0) {
        auto& o = t->entries[prev];
        if (o.pins > 0) o.state = LML_STATE_RETIRING;
        else o.live = false;
    }
    return LML_OK;
}

lml_status lml_pin(lml_table* t, int slot)
{
    if (!t) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    if (slot < 0 || slot >= t->max_slots || !t->entries[slot].live) return LML_ERR_BAD_SLOT;
    ++t->entries[slot].pins;
    return LML_OK;
}

lml_status lml_unpin(lml_table* t, int slot)
{
    if (!t) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    if (slot < 0 || slot >= t->max_slots || !t->entries[slot].live) return LML_ERR_BAD_SLOT;
    auto& e = t->entries[slot];
    if (e.pins <= 0) return LML_ERR_INVALID_ARG;
    if (--e.pins == 0 && e.state == LML_STATE_RETIRING) e.live = false;   // the last work bound to a replaced version has ended
    return LML_OK;
}

lml_status lml_resolve(const lml_table* t, int adapter_id, int* slot_out, int* version_out)
{
    if (!t) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    for (int i = 0; i < t->max_slots; ++i) {
        const auto& e = t->entries[i];
        if (e.live && e.adapter_id == adapter_id && e.state == LML_STATE_SERVING) {
            if (slot_out) *slot_out = i;
            if (version_out) *version_out = e.version;
            return LML_OK;
        }
    }
    return LML_ERR_NOT_FOUND;
}

lml_status lml_slot_state(const lml_table* t, int slot, int* state_out, int* pins_out)
{
    if (!t) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    if (slot < 0 || slot >= t->max_slots || !t->entries[slot].live) return LML_ERR_BAD_SLOT;
    if (state_out) *state_out = t->entries[slot].state;
    if (pins_out) *pins_out = t->entries[slot].pins;
    return LML_OK;
}

lml_status lml_lookup(const lml_table* t, int adapter_id, int version, int* slot_out)
{
    if (!t || !slot_out) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    for (int i = 0; i < t->max_slots; ++i) {
        const auto& e = t->entries[i];
        if (e.live && e.adapter_id == adapter_id && e.version == version) { *slot_out = i; return LML_OK; }
    }
    return LML_ERR_NOT_FOUND;
}

lml_status lml_slot_info(const lml_table* t, int slot, int* adapter_id, int* version, int* rank, float* scale)
{
    if (!t) return LML_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(t->mu);
    if (slot < 0 || slot >= t->max_slots || !t->entries[slot].live) return LML_ERR_BAD_SLOT;
    const auto& e = t->entries[slot];
    if (adapter_id) *adapter_id = e.adapter_id;
    if (version) *version = e.version;
    if (rank) *rank = e.rank;
    if (scale) *scale = e.scale;
    return LML_OK;
}

size_t lml_workspace_bytes(const lml_table* t, int max_tokens, int max_segments)
{
    if (!t || max_tokens < 0 || max_segments < 0 || max_tokens > kMaxTokens) return 0;
    return ws_layout(t, max_tokens, max_segments).total;
}

static lml_status segment_tokens_impl(lml_table* t, const int32_t* ids, int T, int32_t* perm, int32_t* seg_offsets,
                                      int32_t* seg_slot_ids, void* stream, bool by_adapter)
{
    if (!t || T < 0 || T > kMaxTokens || !seg_offsets || !seg_slot_ids || (T > 0 && (!ids || !perm)))
        return LML_ERR_INVALID_ARG;
    const SlotSnapshot snap = snapshot_locked(t);
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    if (launch_segment_tokens(t->arena, snap, ids, T, perm, seg_offsets, seg_slot_ids, (cudaStream_t)stream, by_adapter) !=
        cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    t->last_launches = 1;
    return LML_OK;
}

lml_status lml_segment_tokens(lml_table* t, const int32_t* token_slots, int T, int32_t* perm, int32_t* seg_offsets,
                              int32_t* seg_slot_ids, void* stream)
{
    return segment_tokens_impl(t, token_slots, T, perm, seg_offsets, seg_slot_ids, stream, false);
}

lml_status lml_segment_tokens_adapters(lml_table* t, const int32_t* token_adapter_ids, int T, int32_t* perm,
                                       int32_t* seg_offsets, int32_t* seg_slot_ids, void* stream)
{
    return segment_tokens_impl(t, token_adapter_ids, T, perm, seg_offsets, seg_slot_ids, stream, true);
}

lml_status lora_mixed_linear(lml_table* t, const void* x, const void* W0, int T, const int32_t* seg_offsets,
                             const int32_t* slot_ids, int G, const int32_t* perm, void* y, void* workspace,
                             size_t workspace_bytes, void* stream_v)
{
    if (!t || T < 0 || G < 0 || T > kMaxTokens || G > kMaxTokens) return LML_ERR_INVALID_ARG;
    if (T == 0) { t->last_launches = 0; return LML_OK; }
    if (!x || !W0 || !y || !aligned16(x) || !aligned16(W0) || !aligned16(y)) return LML_ERR_INVALID_ARG;
    if (G > 0 && (!seg_offsets || !slot_ids)) return LML_ERR_INVALID_ARG;
    if (G == 0) perm = nullptr;   // without adapters the row order is irrelevant
    const WsLayout ws = ws_layout(t, T, G);
    const bool decode = T <= kDecodeMaxT;
    const size_t need = decode ? ws.xg_off : (perm ? ws.total : ws.xg_off);
    const bool need_ws = G > 0 || (!decode && perm);
    if (need_ws && (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need))
        return LML_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    const SlotSnapshot snap = snapshot_locked(t);
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    uint8_t* wsb = static_cast<uint8_t*>(workspace);
    int launches = 0;
    cudaError_t e = cudaSuccess;

    if (decode) {
        DecodeArgs a;
        a.x = x; a.W0 = W0; a.y = y; a.perm = perm; a.seg_offsets = seg_offsets; a.slot_ids = slot_ids;
        a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = G; a.num_sms = t->num_sms;
        e = launch_decode(t->arena, snap, a, stream, &launches);
    } else {
        const void* xg = x;
        int32_t* tile_identity = nullptr;
        if (perm) {
            tile_identity = reinterpret_cast<int32_t*>(wsb + ws.ident_off);
            e = launch_gather_rows(x, perm, T, t->d_in, wsb + ws.xg_off, tile_identity, true, t->arena.status, stream);
            if (e == cudaSuccess) { ++launches; xg = wsb + ws.xg_off; }
        }
        PlanWord* plan = reinterpret_cast<PlanWord*>(wsb + ws.plan_off);
        __nv_bfloat16* u_blocks = reinterpret_cast<__nv_bfloat16*>(wsb + ws.u_off);
        // With whole-K tiles the shrink runs inside the GEMM kernel (on the CTAs that own the fewest tiles, ahead of
        // their tiles); otherwise a shrink kernel goes first and the GEMM is its programmatic dependent.
        const bool fused = G > 0 && t->fuse_shrink &&
                           gemm_can_fuse_shrink(T, t->d_in, t->d_out, G, t->num_sms, t->split_bn, t->split_s);
        if (e == cudaSuccess && G > 0 && !fused) {
            e = launch_shrink_pieces(t->arena, snap, xg, T, t->d_in, seg_offsets, slot_ids, G, x, tile_identity, plan,
                                     u_blocks, stream, perm ? 2 : 0);
            if (e == cudaSuccess) ++launches;
        }
        if (e == cudaSuccess) {
            GemmArgs a;
            a.fused_shrink = fused;
            a.x = xg; a.x_in_place = x; a.tile_identity = tile_identity; a.W0 = W0; a.y = y; a.perm = perm; a.seg_offsets = seg_offsets; a.slot_ids = slot_ids;
            a.plan = plan; a.u_blocks = u_blocks ? u_blocks : reinterpret_cast<const __nv_bfloat16*>(x);
            a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = G; a.num_sms = t->num_sms;
            a.overlap_with_previous = G > 0;
            a.split_bn = t->split_bn; a.split_s = t->split_s;
            if (G == 0) a.u_blocks = reinterpret_cast<const __nv_bfloat16*>(W0);   // never read; map needs a valid base
            e = launch_gemm_sm100(t->arena, snap, t->tmap_B256, t->tmap_B128, t->tmap_A, &t->tmaps, a, stream);
            if (e == cudaSuccess) ++launches;
        }
    }
    t->last_launches = launches;
    if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
    return LML_OK;
}

// Segments of a token-form call: one per slot and one for "none" on the grouped path; on the path that keeps the
// tokens in their order, one per slot and row tile at most, and one more.
static int tokens_segments(const lml_table* t, int T)
{
    if (T > t->one_tile_tokens) return t->max_slots + 1;
    return ((T + kTileM - 1) / kTileM) * t->max_slots + 1;
}

size_t lml_tokens_workspace_bytes(const lml_table* t, int max_tokens)
{
    if (!t || max_tokens < 0 || max_tokens > kMaxTokens) return 0;
    // (the largest of the layouts that a call of up to max_tokens tokens can take)
    size_t best = 0;
    const int candidates[2] = {max_tokens, max_tokens < t->one_tile_tokens ? max_tokens : t->one_tile_tokens};
    for (int T : candidates) {
        const int G = tokens_segments(t, T);
        size_t n = ws_layout(t, T, G).total;
        n += round_up((size_t)T * 4 + 4, 1024);               // perm
        n += 2 * round_up((size_t)(G + 1) * 4, 1024);         // seg_offsets, seg_slot_ids
        best = n > best ? n : best;
    }
    return best;
}

size_t lml_dual_workspace_bytes(const lml_table* t, int max_tokens, int max_segments)
{
    if (!t || max_tokens < 0 || max_segments < 0 || max_tokens > kMaxTokens) return 0;
    return ws_layout(t, max_tokens, max_segments, 3).total;
}

lml_status lora_mixed_linear_dual(lml_table* t, const void* x, const void* W0, int T, const int32_t* seg_offsets,
                                  const int32_t* slot_ids_a, const int32_t* slot_ids_b, int G, const int32_t* perm,
                                  void* y_a, void* y_b, void* workspace, size_t workspace_bytes, void* stream_v)
{
    if (!t || T < 0 || G < 1 || T > kMaxTokens || G > kMaxTokens) return LML_ERR_INVALID_ARG;
    if (T == 0) { t->last_launches = 0; return LML_OK; }
    if (!x || !W0 || !y_a || !y_b || y_a == y_b || !seg_offsets || !slot_ids_a || !slot_ids_b || !aligned16(x) ||
        !aligned16(W0) || !aligned16(y_a) || !aligned16(y_b))
        return LML_ERR_INVALID_ARG;
    if (T <= kDecodeMaxT) {
        // One launch of the decode kernel with the two bindings as two projections over the same W0: half of the CTAs
        // per binding, each half exactly a single call (so y_a and y_b are bit for bit those of two calls).  The two
        // halves walk the same rows of W0 at the same time, so the second reader of a line finds it in L2.
        const WsLayout ws1 = ws_layout(t, T, G);
        if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < ws1.xg_off) return LML_ERR_WORKSPACE;
        const SlotSnapshot snap = snapshot_locked(t);
        DeviceGuard guard(t->device);
        if (!guard.ok) return LML_ERR_CUDA;
        SlotSnapshot snaps[2] = {snap, snap};
        const Arena* ars[2] = {&t->arena, &t->arena};
        DecodeArgs args[2];
        for (int p = 0; p < 2; ++p) {
            DecodeArgs& a = args[p];
            a.x = x; a.W0 = W0; a.y = p == 0 ? y_a : y_b; a.perm = perm; a.seg_offsets = seg_offsets;
            a.slot_ids = p == 0 ? slot_ids_a : slot_ids_b;
            a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = G; a.num_sms = t->num_sms;
        }
        const cudaError_t e = launch_decode_multi(ars, snaps, args, 2, (cudaStream_t)stream_v);
        t->last_launches = e == cudaSuccess ? 1 : 0;
        if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
        return LML_OK;
    }
    const WsLayout ws = ws_layout(t, T, G, 3);
    const size_t need = perm ? ws.total : ws.xg_off;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need) return LML_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    const SlotSnapshot snap = snapshot_locked(t);
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    uint8_t* wsb = static_cast<uint8_t*>(workspace);
    int launches = 0;
    cudaError_t e = cudaSuccess;
    const void* xg = x;
    int32_t* tile_identity = nullptr;
    if (perm) {
        tile_identity = reinterpret_cast<int32_t*>(wsb + ws.ident_off);
        e = launch_gather_rows(x, perm, T, t->d_in, wsb + ws.xg_off, tile_identity, true, t->arena.status, stream);
        if (e == cudaSuccess) { ++launches; xg = wsb + ws.xg_off; }
    }
    PlanWord* plan = reinterpret_cast<PlanWord*>(wsb + ws.plan_off);
    __nv_bfloat16* u_blocks = reinterpret_cast<__nv_bfloat16*>(wsb + ws.u_off);
    const size_t num_m = (size_t)(T + kTileM - 1) / kTileM;
    const size_t set_elems = (num_m + (size_t)G) * kTileM * kRankPad;
    // three sets of u blocks: scale.x.A^T under the first slots (set 0) and its negation (set 2), written by
    // one shrink pass, and under the second slots (set 1), by a second pass that runs beside the first:
    // the second output is the first accumulator plus (second delta - first delta)
    e = launch_shrink_pieces(t->arena, snap, xg, T, t->d_in, seg_offsets, slot_ids_a, G, x, tile_identity, plan, u_blocks,
                             stream, false, u_blocks + 2 * set_elems);
    if (e == cudaSuccess) {
        ++launches;
        e = launch_shrink_pieces(t->arena, snap, xg, T, t->d_in, seg_offsets, slot_ids_b, G, x, tile_identity, plan,
                                 u_blocks + set_elems, stream, true);
        if (e == cudaSuccess) ++launches;
    }
    if (e == cudaSuccess) {
        GemmArgs a;
        a.x = xg; a.x_in_place = x; a.tile_identity = tile_identity; a.W0 = W0; a.y = y_a; a.perm = perm;
        a.seg_offsets = seg_offsets; a.slot_ids = slot_ids_a; a.slot_ids2 = slot_ids_b; a.y2 = y_b;
        a.plan = plan; a.u_blocks = u_blocks;
        a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = G; a.num_sms = t->num_sms;
        a.overlap_with_previous = true;
        a.split_bn = t->split_bn; a.split_s = t->split_s;   // (few tokens: the split-K kernel, both bindings' accumulators side by side)
        e = launch_gemm_sm100(t->arena, snap, t->tmap_B256, t->tmap_B128, t->tmap_A, &t->tmaps, a, stream);
        if (e == cudaSuccess) ++launches;
    }
    t->last_launches = launches;
    if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
    return LML_OK;
}

size_t lml_backward_workspace_bytes(const lml_table* t, int max_tokens, int max_segments)
{
    if (!t || max_tokens < 0 || max_segments < 0 || max_tokens > kMaxTokens) return 0;
    return ws_layout(t, max_tokens, max_segments, 2).xg_off;
}

lml_status lora_mixed_linear_backward_adapters(lml_table* t, lml_table* t_T, const void* x, const void* dy, int T,
                                               const int32_t* seg_offsets, const int32_t* slot_ids,
                                               const int32_t* slot_ids_T, int G, float* dA, float* dB, void* workspace,
                                               size_t workspace_bytes, void* stream_v)
{
    if (!t || !t_T || T < 0 || G < 1 || T > kMaxTokens || G > kMaxTokens) return LML_ERR_INVALID_ARG;
    if (t_T->d_in != t->d_out || t_T->d_out != t->d_in || t_T->device != t->device) return LML_ERR_INVALID_ARG;
    if (T == 0) { t->last_launches = 0; return LML_OK; }
    if (!x || !dy || !seg_offsets || !slot_ids || !slot_ids_T || !dA || !dB || !aligned16(x) || !aligned16(dy) ||
        !aligned16(dA) || !aligned16(dB))
        return LML_ERR_INVALID_ARG;
    const WsLayout ws = ws_layout(t, T, G, 2);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < ws.xg_off) return LML_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    const SlotSnapshot snap = snapshot_locked(t);
    const SlotSnapshot snap_T = snapshot_locked(t_T);
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    uint8_t* wsb = static_cast<uint8_t*>(workspace);
    PlanWord* plan = reinterpret_cast<PlanWord*>(wsb + ws.plan_off);
    __nv_bfloat16* u_blocks = reinterpret_cast<__nv_bfloat16*>(wsb + ws.u_off);
    const size_t num_m = (size_t)(T + kTileM - 1) / kTileM;
    const size_t set_elems = (num_m + (size_t)G) * kTileM * kRankPad;
    int launches = 0;
    // set 0: scale.(x.A^T) per position (the forward shrink); set 1: scale.(dy.B), the same pass on the
    // transposed table, whose "A" is B^T
    cudaError_t e = launch_shrink_pieces(t->arena, snap, x, T, t->d_in, seg_offsets, slot_ids, G, x, nullptr, plan, u_blocks, stream);
    if (e == cudaSuccess) {
        ++launches;
        // (a further pass of the same call: it runs beside the first)
        e = launch_shrink_pieces(t_T->arena, snap_T, dy, T, t_T->d_in, seg_offsets, slot_ids_T, G, dy, nullptr, plan,
                                 u_blocks + set_elems, stream, 1);
    }
    if (e == cudaSuccess) {
        ++launches;
        // dA_s[j][k] += sum_t scale.(dy.B)[t][j] x[t][k];   dB_s[n][j] += sum_t dy[t][n] scale.(x.A^T)[t][j]: one launch
        e = launch_weight_grad(snap, u_blocks + set_elems, x, T, t->d_in, seg_offsets, slot_ids, G, dA, 0, stream,
                               u_blocks, dy, t->d_out, dB, 1);
    }
    if (e == cudaSuccess) ++launches;
    t->last_launches = launches;
    if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
    return LML_OK;
}

static lml_status tokens_impl(lml_table* t, const void* x, const void* W0, int T, const int32_t* token_slots, void* y,
                              void* workspace, size_t workspace_bytes, void* stream_v, bool by_adapter)
{
    if (!t || T < 0 || T > kMaxTokens) return LML_ERR_INVALID_ARG;
    if (T == 0) { t->last_launches = 0; return LML_OK; }
    if (!x || !W0 || !y || !token_slots || !aligned16(x) || !aligned16(W0) || !aligned16(y)) return LML_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < lml_tokens_workspace_bytes(t, T))
        return LML_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    uint8_t* wsb = static_cast<uint8_t*>(workspace);
    if (T <= kDecodeMaxT) {
        // Up to 16 tokens need no grouping: the decode kernel handles every row of x on its own, so it reads
        // the slot ids directly.  One launch.
        const SlotSnapshot snap = snapshot_locked(t);
        DeviceGuard guard(t->device);
        if (!guard.ok) return LML_ERR_CUDA;
        const WsLayout ws = ws_layout(t, T, 1);
        DecodeArgs a;
        a.x = x; a.W0 = W0; a.y = y; a.perm = nullptr; a.seg_offsets = nullptr; a.slot_ids = nullptr;
        a.token_slots = token_slots;
        a.by_adapter = by_adapter;
        a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = 1; a.num_sms = t->num_sms;
        int launches = 0;
        const cudaError_t e = launch_decode(t->arena, snap, a, stream, &launches);
        t->last_launches = launches;
        if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
        return LML_OK;
    }
    // (measured on B200 against the one-tile path below, us per call at 20 / 32 / 48 / 64 tokens: 4096 x 4096 13.3 / 13.8 /
    // 19.8 / 24.1 against 19.1 / 20.1 / 20.6 / 20.6; 11008 x 4096 33.5 / 31.5 against 29.2 / 29.7; 4096 x 11008 31.4 / 32.0
    // against 27.4 / 35.4: every block's CTAs take all of W0 in from L2, which a wide output pays for at once)
    const bool small_layer = (long long)t->d_in * t->d_out <= (1ll << 24);
    const int block_limit = t->dec_block_tokens >= 0 ? t->dec_block_tokens
                                                     : (small_layer ? 3 : (t->d_in > 4096 ? 2 : 1)) * kDecodeMaxT;
    if (T <= block_limit) {
        // A few blocks of 16 tokens: one launch of the decode kernel with the blocks as its parts, an equal share of the
        // CTAs each.  The shares walk W0 together, so a line leaves HBM once and the other readers find it in L2; no
        // grouping, no row copy, no shrink kernel.  Every row's arithmetic is that of a decode call.
        const SlotSnapshot snap = snapshot_locked(t);
        DeviceGuard guard(t->device);
        if (!guard.ok) return LML_ERR_CUDA;
        const WsLayout ws = ws_layout(t, T, 1);
        const int nb = (T + kDecodeMaxT - 1) / kDecodeMaxT;
        SlotSnapshot snaps[kDecMaxBlocks];
        DecodeArgs args[kDecMaxBlocks];
        const Arena* ars[kDecMaxBlocks];
        for (int bi = 0; bi < nb; ++bi) {
            snaps[bi] = snap;
            ars[bi] = &t->arena;
            DecodeArgs& a = args[bi];
            const int t0 = bi * kDecodeMaxT;
            a.x = static_cast<const __nv_bfloat16*>(x) + (size_t)t0 * t->d_in;
            a.W0 = W0;
            a.y = static_cast<__nv_bfloat16*>(y) + (size_t)t0 * t->d_out;
            a.perm = nullptr; a.seg_offsets = nullptr; a.slot_ids = nullptr;
            a.token_slots = token_slots + t0;
            a.by_adapter = by_adapter;
            a.T = T - t0 < kDecodeMaxT ? T - t0 : kDecodeMaxT;
            a.d_in = t->d_in; a.d_out = t->d_out; a.G = 1; a.num_sms = t->num_sms;
        }
        const cudaError_t e = launch_decode_multi(ars, snaps, args, nb, stream);
        t->last_launches = e == cudaSuccess ? 1 : 0;
        if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
        return LML_OK;
    }
    // Prefill: the segmentation pass writes perm and the segment arrays behind the layer's own workspace,
    // and the layer call follows on the same stream.
    const int G = tokens_segments(t, T);
    const size_t base = ws_layout(t, T, G).total;
    int32_t* perm = reinterpret_cast<int32_t*>(wsb + base);
    int32_t* seg_offsets = reinterpret_cast<int32_t*>(wsb + base + round_up((size_t)T * 4 + 4, 1024));
    int32_t* seg_ids = seg_offsets + round_up((size_t)(G + 1) * 4, 1024) / 4;
    if (T <= t->one_tile_tokens) {
        // One row tile: the tokens stay where they are.  One launch binds them and writes, per distinct slot of the
        // batch, a block of u whose rows are the slot's tokens (zeros elsewhere); the GEMM then adds block x B per
        // slot.  No grouping, no row copy: two launches instead of four (21 against 30 us at 128 tokens on 4096 x 4096,
        // 32 against 41 on 11008 x 4096, 38 against 46 on 4096 x 11008).
        const SlotSnapshot snap = snapshot_locked(t);
        DeviceGuard guard(t->device);
        if (!guard.ok) return LML_ERR_CUDA;
        const WsLayout ws = ws_layout(t, T, G);
        PlanWord* plan = reinterpret_cast<PlanWord*>(wsb + ws.plan_off);
        __nv_bfloat16* u_blocks = reinterpret_cast<__nv_bfloat16*>(wsb + ws.u_off);
        int launches = 0;
        cudaError_t e = launch_bind_shrink_tile(t->arena, snap, token_slots, T, t->d_in, x, seg_offsets, seg_ids, G, plan,
                                                u_blocks, t->bind_threads > 0 ? t->bind_threads : (t->d_in > 4096 ? 1024 : 512), stream, by_adapter);
        if (e == cudaSuccess) {
            ++launches;
            GemmArgs a;
            a.fused_shrink = false;
            a.x = x; a.x_in_place = x; a.tile_identity = nullptr; a.W0 = W0; a.y = y; a.perm = nullptr;
            a.seg_offsets = seg_offsets; a.slot_ids = seg_ids;
            a.plan = plan; a.u_blocks = u_blocks;
            a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = G; a.num_sms = t->num_sms;
            a.overlap_with_previous = true;
            a.split_bn = t->split_bn; a.split_s = t->split_s;
            e = launch_gemm_sm100(t->arena, snap, t->tmap_B256, t->tmap_B128, t->tmap_A, &t->tmaps, a, stream);
            if (e == cudaSuccess) ++launches;
        }
        t->last_launches = launches;
        if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
        return LML_OK;
    }
    lml_status st = segment_tokens_impl(t, token_slots, T, perm, seg_offsets, seg_ids, stream_v, by_adapter);
    if (st != LML_OK) return st;
    st = lora_mixed_linear(t, x, W0, T, seg_offsets, seg_ids, G, perm, y, workspace, base, stream_v);
    if (st == LML_OK) t->last_launches += 1;
    return st;
}

lml_status lora_mixed_linear_tokens(lml_table* t, const void* x, const void* W0, int T, const int32_t* token_slots,
                                    void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return tokens_impl(t, x, W0, T, token_slots, y, workspace, workspace_bytes, stream, false);
}

lml_status lora_mixed_linear_adapters(lml_table* t, const void* x, const void* W0, int T,
                                      const int32_t* token_adapter_ids, void* y, void* workspace,
                                      size_t workspace_bytes, void* stream)
{
    return tokens_impl(t, x, W0, T, token_adapter_ids, y, workspace, workspace_bytes, stream, true);
}

size_t lml_multi_workspace_bytes(lml_table* const* tables, int P, int max_tokens)
{
    if (!tables || P < 1 || P > LML_MAX_PROJECTIONS || max_tokens < 0 || max_tokens > kMaxTokens) return 0;
    size_t n = 0;
    for (int p = 0; p < P; ++p) {
        if (!tables[p]) return 0;
        const size_t b = lml_tokens_workspace_bytes(tables[p], max_tokens);
        n = b > n ? b : n;
    }
    return n;
}

lml_status lora_mixed_linear_multi(lml_table* const* tables, int P, const void* x, const void* const* W0, int T,
                                   const int32_t* const* token_slots, void* const* y, void* workspace,
                                   size_t workspace_bytes, void* stream_v)
{
    if (!tables || !W0 || !token_slots || !y || P < 1 || P > LML_MAX_PROJECTIONS || T < 0 || T > kMaxTokens) return LML_ERR_INVALID_ARG;
    for (int p = 0; p < P; ++p) {
        if (!tables[p] || tables[p]->d_in != tables[0]->d_in || tables[p]->device != tables[0]->device) return LML_ERR_INVALID_ARG;
        for (int q = 0; q < p; ++q) if (y[q] == y[p] && T > 0) return LML_ERR_INVALID_ARG;
    }
    if (T == 0) { for (int p = 0; p < P; ++p) tables[p]->last_launches = 0; return LML_OK; }
    if (!x || !aligned16(x)) return LML_ERR_INVALID_ARG;
    for (int p = 0; p < P; ++p)
        if (!W0[p] || !y[p] || !token_slots[p] || !aligned16(W0[p]) || !aligned16(y[p])) return LML_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < lml_multi_workspace_bytes(tables, P, T))
        return LML_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    bool distinct = true;   // (a table's counters serve one projection of a launch)
    for (int p = 0; p < P; ++p)
        for (int q = 0; q < p; ++q) distinct = distinct && tables[p] != tables[q];
    const int nb = 1;   // (projections times blocks of 16 tokens in one launch was measured: 44.1 us against 42.8 us for q/k/v at 32 tokens as one call per projection)
    if (P > 1 && distinct && T <= kDecodeMaxT) {
        // One launch of the decode kernel for all projections: its CTAs are dealt out over them, each works on its
        // projection as in a call of its own, and the fixed costs of a call are paid once.
        DeviceGuard guard(tables[0]->device);
        if (!guard.ok) return LML_ERR_CUDA;
        SlotSnapshot snaps[kDecMaxBlocks];
        DecodeArgs args[kDecMaxBlocks];
        const Arena* ars[kDecMaxBlocks];
        const WsLayout ws = ws_layout(tables[0], T, 1);
        int n = 0;
        for (int p = 0; p < P; ++p) {
            const SlotSnapshot snap = snapshot_locked(tables[p]);
            for (int bi = 0; bi < nb; ++bi, ++n) {
                const int t0 = bi * kDecodeMaxT;
                snaps[n] = snap;
                ars[n] = &tables[p]->arena;
                DecodeArgs& a = args[n];
                a.x = static_cast<const __nv_bfloat16*>(x) + (size_t)t0 * tables[0]->d_in;
                a.W0 = W0[p];
                a.y = static_cast<__nv_bfloat16*>(y[p]) + (size_t)t0 * tables[p]->d_out;
                a.perm = nullptr; a.seg_offsets = nullptr; a.slot_ids = nullptr;
                a.token_slots = token_slots[p] + t0;
                a.by_adapter = false;
                a.T = T - t0 < kDecodeMaxT ? T - t0 : kDecodeMaxT;
                a.d_in = tables[0]->d_in; a.d_out = tables[p]->d_out; a.G = 1; a.num_sms = tables[0]->num_sms;
            }
        }
        const cudaError_t e = launch_decode_multi(ars, snaps, args, n, stream);
        if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
        for (int p = 0; p < P; ++p) tables[p]->last_launches = p == 0 ? 1 : 0;
        return LML_OK;
    }
    // one projection after the other: larger batches (the GEMM path), a single projection, or a table named twice
    for (int p = 0; p < P; ++p) {
        const lml_status st = tokens_impl(tables[p], x, W0[p], T, token_slots[p], y[p], workspace, workspace_bytes, stream_v, false);
        if (st != LML_OK) return st;
    }
    return LML_OK;
}

size_t lml_host_workspace_bytes(const lml_table* t, int max_tokens, int max_segments)
{
    if (!t || max_tokens < 0 || max_segments < 0 || max_tokens > kMaxTokens) return 0;
    size_t n = ws_layout(t, max_tokens, max_segments).total;
    n += round_up((size_t)max_tokens * t->d_in * 2, 1024);    // x staging
    n += round_up((size_t)max_tokens * t->d_out * 2, 1024);   // y staging
    n += round_up((size_t)(max_segments + 1) * 4, 1024) + round_up((size_t)max_segments * 4 + 4, 1024);
    n += round_up((size_t)max_tokens * 4 + 4, 1024);          // perm staging
    n += lml_table::kHostChunks * round_up((size_t)(2 * max_segments + 2) * 4, 256);   // per-chunk segment arrays
    return n;
}

lml_status lora_mixed_linear_host(lml_table* t, const void* x_host, const void* W0, int T,
                                  const int32_t* seg_offsets_host, const int32_t* slot_ids_host, int G,
                                  const int32_t* perm_host, void* y_host, void* workspace, size_t workspace_bytes,
                                  void* stream_v)
{
    if (!t || T < 0 || G < 0 || T > kMaxTokens || G > kMaxTokens) return LML_ERR_INVALID_ARG;
    if (T == 0) { t->last_launches = 0; return LML_OK; }
    if (!x_host || !W0 || !y_host || (G > 0 && (!seg_offsets_host || !slot_ids_host))) return LML_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < lml_host_workspace_bytes(t, T, G))
        return LML_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    uint8_t* p = static_cast<uint8_t*>(workspace);
    const size_t inner = ws_layout(t, T, G).total;
    uint8_t* xs = p + inner;
    uint8_t* ys = xs + round_up((size_t)T * t->d_in * 2, 1024);
    uint8_t* so = ys + round_up((size_t)T * t->d_out * 2, 1024);
    uint8_t* si = so + round_up((size_t)(G + 1) * 4, 1024);
    uint8_t* pm = si + round_up((size_t)G * 4 + 4, 1024);
    // Decode calls on pinned buffers: no DMA copies.  One kernel pulls the inputs out of host memory, and
    // the decode kernel writes y straight into the caller's buffer.  (Anything else: copies, below.)
    if (T <= kDecodeMaxT) {
        auto device_view = [](const void* h, size_t align) -> void* {
            if (!h) return nullptr;
            cudaPointerAttributes a;
            if (cudaPointerGetAttributes(&a, h) != cudaSuccess) { cudaGetLastError(); return nullptr; }
            if (a.type != cudaMemoryTypeHost || !a.devicePointer) return nullptr;
            return (reinterpret_cast<uintptr_t>(a.devicePointer) & (align - 1)) ? nullptr : a.devicePointer;
        };
        void* xd = device_view(x_host, 16);
        void* yd = device_view(y_host, 16);
        void* sod = G > 0 ? device_view(seg_offsets_host, 4) : nullptr;
        void* sid = G > 0 ? device_view(slot_ids_host, 4) : nullptr;
        void* pmd = perm_host ? device_view(perm_host, 4) : nullptr;
        if (xd && yd && (G == 0 || (sod && sid)) && (!perm_host || pmd)) {
            if (launch_stage_host_inputs(xd, xs, (size_t)T * t->d_in * 2, (const int32_t*)sod, reinterpret_cast<int32_t*>(so),
                                         G > 0 ? G + 1 : 0, (const int32_t*)sid, reinterpret_cast<int32_t*>(si), G,
                                         (const int32_t*)pmd, reinterpret_cast<int32_t*>(pm), perm_host ? T : 0,
                                         stream) != cudaSuccess) {
                cudaGetLastError();
                return LML_ERR_CUDA;
            }
            lml_status st = lora_mixed_linear(t, xs, W0, T, reinterpret_cast<int32_t*>(so), reinterpret_cast<int32_t*>(si), G,
                                              perm_host ? reinterpret_cast<int32_t*>(pm) : nullptr, yd, p, inner, stream);
            if (st == LML_OK) t->last_launches += 1;
            return st;
        }
    }
    // Large calls on pinned buffers, rows in segment order: in chunks of whole row tiles, the copy of the next
    // chunk's x, the layer on this chunk and the copy of the last chunk's y side by side on three streams
    // (the caller's and two of the table's), joined again before the call's last operation.
    constexpr int kChunks = lml_table::kHostChunks;
    if (T >= 256 * kChunks && !perm_host) {
        auto pinned = [](const void* h) {
            cudaPointerAttributes a;
            if (cudaPointerGetAttributes(&a, h) != cudaSuccess) { cudaGetLastError(); return false; }
            return a.type == cudaMemoryTypeHost;
        };
        if (pinned(x_host) && pinned(y_host)) {
            const int rows = (int)round_up((size_t)(T + kChunks - 1) / kChunks, kTileM);
            const int stride = (int)(round_up((size_t)(2 * G + 2) * 4, 256) / 4);
            int32_t* chunk_arrays = reinterpret_cast<int32_t*>(pm + round_up((size_t)T * 4 + 4, 1024));
            bool ok = true;
            int launches = 0;
            if (G > 0) {
                ok = ok && cudaMemcpyAsync(so, seg_offsets_host, (size_t)(G + 1) * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
                ok = ok && cudaMemcpyAsync(si, slot_ids_host, (size_t)G * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
                ok = ok && launch_clip_segments(reinterpret_cast<int32_t*>(so), reinterpret_cast<int32_t*>(si), G, T, rows,
                                                (T + rows - 1) / rows, chunk_arrays, stride, stream) == cudaSuccess;
                ++launches;
            }
            ok = ok && cudaEventRecord(t->ev_begin, stream) == cudaSuccess;        // everything before this call on the caller's stream
            ok = ok && cudaStreamWaitEvent(t->copy_in, t->ev_begin, 0) == cudaSuccess;
            const size_t xrow = (size_t)t->d_in * 2, yrow = (size_t)t->d_out * 2;
            int c = 0;
            for (int r0 = 0; r0 < T && ok; r0 += rows, ++c) {
                const int Tc = T - r0 < rows ? T - r0 : rows;
                ok = ok && cudaMemcpyAsync(xs + r0 * xrow, static_cast<const uint8_t*>(x_host) + r0 * xrow, Tc * xrow,
                                           cudaMemcpyHostToDevice, t->copy_in) == cudaSuccess;
                ok = ok && cudaEventRecord(t->ev_in[c], t->copy_in) == cudaSuccess;
            }
            if (!ok) { cudaGetLastError(); return LML_ERR_CUDA; }
            c = 0;
            for (int r0 = 0; r0 < T; r0 += rows, ++c) {
                const int Tc = T - r0 < rows ? T - r0 : rows;
                if (cudaStreamWaitEvent(stream, t->ev_in[c], 0) != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
                const int32_t* so_c = chunk_arrays + (size_t)c * stride;
                lml_status st = lora_mixed_linear(t, xs + r0 * xrow, W0, Tc, G > 0 ? so_c : nullptr, G > 0 ? so_c + G + 1 : nullptr, G,
                                                  nullptr, ys + r0 * yrow, p, inner, stream);
                if (st != LML_OK) return st;
                launches += t->last_launches;
                ok = ok && cudaEventRecord(t->ev_layer[c], stream) == cudaSuccess;
                ok = ok && cudaStreamWaitEvent(t->copy_out, t->ev_layer[c], 0) == cudaSuccess;
                ok = ok && cudaMemcpyAsync(static_cast<uint8_t*>(y_host) + r0 * yrow, ys + r0 * yrow, Tc * yrow,
                                           cudaMemcpyDeviceToHost, t->copy_out) == cudaSuccess;
                if (!ok) { cudaGetLastError(); return LML_ERR_CUDA; }
            }
            ok = ok && cudaEventRecord(t->ev_done, t->copy_out) == cudaSuccess;
            ok = ok && cudaStreamWaitEvent(stream, t->ev_done, 0) == cudaSuccess;   // the caller's stream ends with y in place
            if (!ok) { cudaGetLastError(); return LML_ERR_CUDA; }
            t->last_launches = launches;
            return LML_OK;
        }
    }
    bool ok = cudaMemcpyAsync(xs, x_host, (size_t)T * t->d_in * 2, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (G > 0) {
        ok = ok && cudaMemcpyAsync(so, seg_offsets_host, (size_t)(G + 1) * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(si, slot_ids_host, (size_t)G * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    }
    if (perm_host)
        ok = ok && cudaMemcpyAsync(pm, perm_host, (size_t)T * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return LML_ERR_CUDA; }
    lml_status st = lora_mixed_linear(t, xs, W0, T, reinterpret_cast<int32_t*>(so), reinterpret_cast<int32_t*>(si), G,
                                      perm_host ? reinterpret_cast<int32_t*>(pm) : nullptr, ys, p, inner, stream);
    if (st != LML_OK) return st;
    if (cudaMemcpyAsync(y_host, ys, (size_t)T * t->d_out * 2, cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
        cudaGetLastError();
        return LML_ERR_CUDA;
    }
    return LML_OK;
}

lml_status lml_device_status(lml_table* t, uint32_t* flags_out, void* stream_v)
{
    if (!t || !flags_out) return LML_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_v;
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;
    uint32_t v = 0;
    bool ok = cudaMemcpyAsync(&v, t->arena.status, sizeof v, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaMemsetAsync(t->arena.status, 0, sizeof v, stream) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    if (ok && (v & LML_FLAG_TIMEOUT)) {
        // a launch gave up on a wait: its counters may have been left behind, so the decode kernel's exchange blocks
        // start over (only then: in normal operation nothing here touches memory that a call in flight uses)
        ok = cudaMemsetAsync(t->arena.dec_u, 0, (size_t)kDecMaxBlocks * kDecExchStride * sizeof(unsigned long long), stream) == cudaSuccess;
        ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    }
    if (!ok) { cudaGetLastError(); return LML_ERR_CUDA; }
    *flags_out = v;
    return LML_OK;
}

int lml_last_launch_count(const lml_table* t) { return t ? t->last_launches : 0; }

}  // extern "C"
