// Host-visible declarations of the streaming decode kernel (lml_decode_stream.cu).  Not part of the public ABI.
#pragma once
#include "lml_internal.cuh"

namespace lml {

constexpr int kDsMaxProj = LML_MAX_PROJECTIONS;   // projections that one decode launch can serve
constexpr int kDsMaxLiveRows = 1024;               // live rows of A (sum of the resident ranks, all projections) the kernel streams at most
constexpr size_t kDsExchangeBytes = (size_t)kDsMaxLiveRows * 16 * sizeof(float);   // u[live row][16 tokens]

// One projection of a decode launch.
struct DsProj {
    const __nv_bfloat16* W0;
    __nv_bfloat16* y;
    const __nv_bfloat16* arenaA;
    const __nv_bfloat16* arenaB;
    const __nv_bfloat16* arenaBc;
    const int32_t* token_slots;   // one id per row of x (tokens form), else null
    const int32_t* adapter_map;   // the ids are adapter ids, resolved through this map; else null
    uint32_t* status;             // the table's sticky flags
    int N;                        // rows of W0 = columns of y
    int pad;
};

struct DsParams {
    DsProj proj[kDsMaxProj];
    const __nv_bfloat16* x;
    float* u;                     // exchange buffer, kDsExchangeBytes: u[live row][16 tokens]
    const int32_t* seg_offsets;   // segments form (one projection only): as lora_mixed_linear
    const int32_t* slot_ids;
    const int32_t* perm;
    unsigned int* sync_words;     // [0] live rows published, [1] CTAs that have signed off (in the first table's status block)
    int P, T, K, G;               // G == 0: no adapters in this call
    int live_rows;                // all projections together; 0 when G == 0
    int n_total;                  // rows of all base weights together
    int patience;                 // clock cycles a CTA waits for its peers' rows before it computes them itself
    int early_adapters;           // 1: rows of A may be fetched before the wait for the preceding work on the stream
};

// Whether the streaming kernel takes a decode call with these tables (else: the kernel of lml_decode.cu, one projection at a time).
bool decode_stream_eligible(const SlotSnapshot* snaps, const int* d_out, int P, int d_in, bool has_adapters, int num_sms);
cudaError_t decode_stream_init();
// snaps[P]: the tables' snapshots.  The grid and the row ranges follow from the parameters.
cudaError_t launch_decode_stream(const SlotSnapshot* snaps, DsParams prm, int num_sms, cudaStream_t stream);

}  // namespace lml
