// gsa_sparse_gated_attn_fwd_static: sparse gated attention for callers that cannot allocate.
//
// The regular entry point keeps V' = bf16(V * sigmoid(g2)) (Eq. 9 as a streaming pre-pass) in a
// workspace the caller allocates.  Some callers have no way to do that: code running inside a
// pre-reserved memory pool, a real-time or signal-handling context, or a host application whose
// allocator must not be entered from the thread that drives the GPU -- for them cudaMalloc (which
// may also synchronise the device) is off limits.  This variant keeps V' in an array that is part
// of the library image itself, so nothing is allocated at any time: not by this call, not by a
// helper library.  The price is a fixed upper size and one shared buffer per GPU.
#include <mutex>
#include <stdio.h>

#include "gsa_common.cuh"

namespace gsa {
namespace {

constexpr size_t kStaticVgBytes = GSA_STATIC_SCRATCH_BYTES;

// Every GPU that loads the library holds this array until the process exits.
// Layout: a 256-byte head holding the device status word, the attention scratch, the gated values.
static __device__ __align__(256) unsigned char g_static_scratch[kStatusBytes + kStaticVgBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};     // device address of g_static_scratch, per device

// In host code `g_static_scratch` is only a handle for the runtime, not an address the GPU can use;
// the address on the current device has to be asked for, once per device.
cudaError_t scratch_on_current_device(void** ptr) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
    }
    *ptr = g_scratch_ptr[dev];
    return cudaSuccess;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

cudaError_t static_scratch_address(void** ptr) { return scratch_on_current_device(ptr); }

}  // namespace gsa

using namespace gsa;

extern "C" int gsa_sparse_gated_attn_fwd_static(const gsa_params_t* p, const void* Q, const void* K,
                                                const void* V, const void* g1_logits, const void* g2_logits,
                                                const int32_t* idx, const int32_t* kt, void* out, void* stream) {
    // parameter checks are those of every other entry point
    size_t unused = 0;
    int rc = gsa_workspace_bytes(p, 0, &unused);
    if (rc) return rc;
    const int qe = p->q_end <= 0 ? p->Lq : p->q_end;
    if (p->q_begin < 0 || p->q_begin >= qe || qe > p->Lq) return GSA_ERR_INVALID_ARG;
    if (!Q || !K || !V || !g1_logits || !g2_logits || !idx || !kt || !out) return GSA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(g1_logits) || !aligned16(g2_logits) ||
        !aligned16(idx) || !aligned16(out))
        return GSA_ERR_INVALID_ARG;

    const size_t vg_bytes = (size_t)p->B * p->Lk * p->n_kv * p->d_h * 2;
    const size_t attn_bytes = (attn_scratch_bytes(*p) + 255) / 256 * 256;
    if (vg_bytes + attn_bytes > kStaticVgBytes) {
        fprintf(stderr,
                "gsa_sparse_gated_attn_fwd_static: %zu bytes of gated values (B*Lk*n_kv*d_h*2) plus %zu bytes of "
                "attention scratch exceed the built-in scratch array of %zu bytes; use "
                "gsa_sparse_gated_attn_fwd with a workspace\n",
                vg_bytes, attn_bytes, kStaticVgBytes);
        return GSA_ERR_STATIC_SCRATCH;
    }

    void* scratch = nullptr;
    cudaError_t e = scratch_on_current_device(&scratch);
    if (e != cudaSuccess) {
        fprintf(stderr, "gsa: CUDA error: %s\n", cudaGetErrorString(e));
        return GSA_ERR_CUDA;
    }
    cudaStream_t st = (cudaStream_t)stream;
    void* attn_scratch = (char*)scratch + kStatusBytes;
    __nv_bfloat16* Vg = (__nv_bfloat16*)((char*)scratch + kStatusBytes + attn_bytes);
    // The array keeps what the previous call left in it.  The status word must start at zero and is
    // cleared here; the pre-pass overwrites every gated value the attention kernel will read, and the
    // attention kernels write every state slot before they read it.
    t_dev_status = (int32_t*)scratch;
    e = cudaMemsetAsync(scratch, 0, kStatusBytes, st);
    if (e == cudaSuccess)
        e = launch_value_gate((const __nv_bfloat16*)V, (const __nv_bfloat16*)g2_logits, Vg,
                          (int64_t)p->B * p->Lk * p->n_kv * p->d_h, st);
    if (e == cudaSuccess) {
        RowRange rr{0, p->B, p->q_begin, qe - p->q_begin};
        IdxLayout il{0, rr.q_begin, rr.R};
        e = launch_sparse_attn(*p, rr, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, Vg,
                               (const __nv_bfloat16*)g1_logits, nullptr, idx, kt, il, (__nv_bfloat16*)out,
                               attn_scratch, st);
    }
    if (e != cudaSuccess) {
        fprintf(stderr, "gsa: CUDA error: %s\n", cudaGetErrorString(e));
        return GSA_ERR_CUDA;
    }
    return GSA_OK;
}
