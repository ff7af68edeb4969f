// lora_mixed_linear_decode_static: the decode form of the layer for callers that cannot hand the
// library any scratch memory.  See the declaration in include/lora_mixed_linear.h.
//
// The decode kernel needs a little scratch between its shrink phase and its epilogue: the exchange
// block through which the CTAs of the grid hand one another the scaled shrink result u[16][64]
// (each fp32 value beside the mark of the launch that wrote it, then three counters).  Here it lives
// in a file-scope device array that is part of the library image: every GPU context that loads the
// library carries these 8448 bytes until the process exits, and nothing is ever allocated or freed.
#include "lml_table.cuh"

using namespace lml;

namespace {

constexpr size_t kStaticU = (size_t)kDecExchStride * sizeof(unsigned long long);   // 8256 bytes
constexpr size_t kStaticScratchBytes = 8448;
static_assert(kStaticU <= kStaticScratchBytes, "static scratch too small");

// In host code this name is only a handle for the runtime, not a device address: the address the
// kernels get is looked up with cudaGetSymbolAddress below, with the table's device current.
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

// Device address of the scratch array on the current device.  Asked of the runtime on every call: the
// lookup allocates nothing and costs little, and an address remembered across a tear-down of the device's
// context (cudaDeviceReset and a new table on the same ordinal) would be stale.
cudaError_t scratch_address(void** out)
{
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_decode_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    *out = p;
    return cudaSuccess;
}

}  // namespace

extern "C" lml_status lora_mixed_linear_decode_static(lml_table* t, const void* x, const void* W0, int T,
                                                      const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                                                      const int32_t* perm, void* y, void* stream_v)
{
    if (!t || T < 0 || G < 0 || G > kMaxTokens) return LML_ERR_INVALID_ARG;
    if (T > kDecodeMaxT) return LML_ERR_TOO_LARGE;   // the static scratch holds 16 token rows, no more
    if (T == 0) { t->last_launches = 0; return LML_OK; }
    if (!x || !W0 || !y || !aligned16(x) || !aligned16(W0) || !aligned16(y)) return LML_ERR_INVALID_ARG;
    if (G > 0 && (!seg_offsets || !slot_ids)) return LML_ERR_INVALID_ARG;
    if (G == 0) perm = nullptr;
    cudaStream_t stream = (cudaStream_t)stream_v;
    const SlotSnapshot snap = snapshot_locked(t);
    DeviceGuard guard(t->device);
    if (!guard.ok) return LML_ERR_CUDA;

    void* scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }

    // The array starts as zeros (a file-scope object) and keeps whatever the previous call left: the
    // block's own mark counter tells this launch's entries from those of earlier ones, whichever table
    // they were for.
    int launches = 0;
    DecodeArgs a;
    a.x = x; a.W0 = W0; a.y = y; a.perm = perm; a.seg_offsets = seg_offsets; a.slot_ids = slot_ids;
    a.exch = static_cast<unsigned long long*>(scratch);
    a.T = T; a.d_in = t->d_in; a.d_out = t->d_out; a.G = G; a.num_sms = t->num_sms;
    cudaError_t e = launch_decode(t->arena, snap, a, stream, &launches);
    t->last_launches = launches;
    if (e != cudaSuccess) { cudaGetLastError(); return LML_ERR_CUDA; }
    return LML_OK;
}
