// The adapter slot table object behind the opaque lml_table handle, shared by the files that
// implement the C ABI.  Not part of the public ABI.
#pragma once
#include <mutex>

#include "lml_internal.cuh"

struct lml_table {
    int device = 0, d_in = 0, d_out = 0, max_slots = 0, num_sms = 0;
    struct Entry {
        bool live = false;
        int adapter_id = 0, version = 0, rank = 0;
        float scale = 0.f;
        int state = 0;   // LML_STATE_*: resident (staged or plain), serving, retiring
        int pins = 0;    // work in flight that is bound to this entry
        uint16_t gen = 0;   // the table's registration counter when the entry was made (see the adapter map)
    } entries[lml::kMaxSlots];
    uint16_t next_gen = 0;
    lml::Arena arena{};
    CUtensorMap tmap_B256, tmap_B128;   // packed B arena as [max_slots][d_out][64], boxes 64 x 256 x 1 and 64 x 128 x 1
    CUtensorMap tmap_A;                 // packed A arena as [max_slots][64][d_in], box 64 x 64 x 1
    bool fuse_shrink = true;            // LML_FUSE_SHRINK=0 when the table was created: always the separate shrink kernel (a test knob)
    lml::TmapCache tmaps;               // tensor maps of the caller's buffers seen so far
    int bind_threads = 0;               // LML_BIND_THREADS as it stood when the table was created (0: the library chooses; a test knob)
    int one_tile_tokens = lml::kTileM;  // token-form calls of up to this many tokens (beyond the decode kernel's range) keep the tokens in their order: one or two row tiles, set when the table is created; LML_ONE_TILE=0 or LML_ONE_TILE_TOKENS=n at that time change it (test knobs)
    int dec_block_tokens = -1;          // token-form calls of up to this many tokens run as blocks of 16 on the decode kernel; -1: the library's own limit (LML_DECODE_BLOCK_TOKENS as it stood when the table was created)
    int split_bn = -1, split_s = -1;    // LML_GEMM_SPLIT as it stood when the table was created (-1: not set)
    // Retiring a serving entry clears its word of the device map with a kernel on a stream; the event marks
    // that point, and every later registration makes its own stream wait for it before it overwrites a slot.
    cudaEvent_t ev_map = nullptr;
    bool map_clear_recorded = false;
    int last_launches = 0;
    // host-buffer form of large calls: the copies of x in and of y out run on two streams of the table's own,
    // chunk by chunk beside the layer (created with the table: the call itself creates nothing)
    static constexpr int kHostChunks = 8;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_begin = nullptr, ev_done = nullptr, ev_in[kHostChunks] = {}, ev_layer[kHostChunks] = {};
    mutable std::mutex mu;
};

namespace lml {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Copy of the live slots' rank and scale, taken under the table's lock.
inline SlotSnapshot snapshot_locked(const lml_table* t)
{
    std::lock_guard<std::mutex> lock(t->mu);
    SlotSnapshot s;
    for (int i = 0; i < kMaxSlots; ++i) {
        const bool live = i < t->max_slots && t->entries[i].live;
        s.rank[i] = live ? (uint8_t)t->entries[i].rank : 0;
        s.scale[i] = live ? t->entries[i].scale : 0.f;
        s.gen[i] = live ? t->entries[i].gen : (uint16_t)0;
    }
    s.max_slots = t->max_slots;
    return s;
}

constexpr int kMaxTokens = kTileM * 32768;   // keeps every grid dimension and int index in range

}  // namespace lml
