// sobek_conv_fwd_static: the forward convolution for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc (or any allocating routine) at the point
// where they run the convolution: code that runs inside another framework's memory plan,
// inside a real-time loop, or in a process whose device memory was handed out completely at
// start-up.  For them this entry point keeps the scratch memory that sobek_conv_fwd takes from
// the caller's workspace (the re-laid-out copy of R, the bounded receiver state of one node
// chunk and the status word) in a fixed array that is part of the library image itself.
#include <algorithm>

#include "internal.h"

using namespace sobek;

namespace {

// The scratch array.  Every GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = size_t(32) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a stand-in for the symbol, not a device address; the
// address has to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace

extern "C" size_t sobek_static_scratch_bytes(void) { return kStaticScratchBytes; }

// The status word of the array on the current device (the kernels' bounded waits and range guards write it).
extern "C" int sobek_static_last_status(void* stream) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices || !g_scratch_addr[dev]) {
        (void)cudaGetLastError();
        return SOBEK_ERR_CUDA;
    }
    int h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, g_scratch_addr[dev], sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return SOBEK_ERR_CUDA; }
    return h;
}

extern "C" int sobek_conv_fwd_static(const sobek_plan* p, const sobek_graph* g, const float* x,
                                     const float* Y, const float* phi, const float* R, float* y,
                                     void* stream) {
    if (!p || !g || g->N < 0 || g->E < 0) return SOBEK_ERR_INVALID_ARG;
    if (g->N >= (int64_t(1) << 31) || g->E >= (int64_t(1) << 31)) return SOBEK_ERR_UNSUPPORTED;
    if (!y || !R || (g->N > 0 && (!x || !g->row_ptr)) || (g->E > 0 && (!Y || !phi || !g->col)))
        return SOBEK_ERR_INVALID_ARG;
    if (p->device < 0) return SOBEK_ERR_CUDA;
    if (p->uvu || p->mul_ir) return SOBEK_ERR_UNSUPPORTED;   // this entry point covers the fully connected mode in ir_mul order only
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return SOBEK_ERR_CUDA;
    }
    if (dev != p->device) return SOBEK_ERR_INVALID_ARG;   // the plan's tables live on the device it was created on
    if ((((uintptr_t)x | (uintptr_t)Y | (uintptr_t)phi | (uintptr_t)R | (uintptr_t)y) & 15) != 0) return SOBEK_ERR_INVALID_ARG;
    if (!g_scratch_addr[dev]) {   // set-up on the first call on this device
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return SOBEK_ERR_CUDA;
        }
        g_scratch_addr[dev] = (unsigned char*)ptr;
    }
    unsigned char* base = g_scratch_addr[dev];
    // layout: [status 256 B][R as bf16 hi, lo][receiver state of one node chunk as bf16 hi, lo]
    const size_t rbytes = align256((size_t)p->fwd.nk_elems * 2);
    const size_t per_node = (size_t)std::max<int64_t>(p->fwd.zb_elems, 1) * 2;   // one of (hi, lo)
    if (kHeaderBytes + 2 * rbytes + 2 * (per_node + 256) > kStaticScratchBytes) return SOBEK_ERR_WORKSPACE;
    const int64_t chunk = std::min<int64_t>(
        std::max<int64_t>(g->N, 1), (int64_t)((kStaticScratchBytes - kHeaderBytes - 2 * rbytes - 512) / (2 * per_node)));
    unsigned char* nkh = base + kHeaderBytes;
    unsigned char* nkl = nkh + rbytes;
    unsigned char* zh = nkl + rbytes;
    unsigned char* zl = zh + align256((size_t)chunk * per_node);
    cudaStream_t s = (cudaStream_t)stream;
#define CKS(expr)                                            \
    do {                                                     \
        if ((expr) != cudaSuccess) {                         \
            (void)cudaGetLastError();                        \
            return SOBEK_ERR_CUDA;                           \
        }                                                    \
    } while (0)
    // the array keeps whatever the previous call left: the status word must start at zero
    CKS(cudaMemsetAsync(base, 0, kHeaderBytes, s));
    if (g->N == 0) return SOBEK_OK;
    bool uncovered = false;
    for (const DGroup& G : p->fwd.groups) uncovered = uncovered || (G.path_end == G.path_begin);
    if (g->E == 0 || uncovered) CKS(launch_fill_zero(y, g->N * (int64_t)p->C_y, s));
    if (g->E == 0) return SOBEK_OK;
    CKS(launch_pack_R_bf16(p, p->fwd, 0, 1, R, nkh, nkl, s));
    const EdgeView rv{g->row_ptr, nullptr, g->col, g->row_ptr, g->N, g->E, 0};
    const Direction& dir = p->fwd;
    for (int64_t n0 = 0; n0 < g->N; n0 += chunk) {
        const int64_t nn = std::min(chunk, g->N - n0);
        // every element of the chunk's state that the contraction reads is overwritten first
        CKS(launch_stream(p, dir, rv, n0, nn, x, nullptr, SplitSrc{}, Y, nullptr, phi, nullptr, 0, zh, zl, (int*)base, s));
        for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
            const DGroup& G = dir.groups[gi];
            if (G.path_end == G.path_begin) continue;
            const uint16_t* ah = (const uint16_t*)zh + nn * dir.zb_off[gi];
            const uint16_t* al = (const uint16_t*)zl + nn * dir.zb_off[gi];
            CKS(launch_gemm_tc(ah, al, dir.nk_ld[gi], (const uint16_t*)nkh + dir.nk_off[gi],
                               (const uint16_t*)nkl + dir.nk_off[gi], dir.nk_ld[gi],
                               y + n0 * dir.C_dst + G.dst_off, dir.C_dst, G.c_dst, G.d_dst, nn * G.d_dst, G.c_dst,
                               G.D, 0, 0, (int*)base, s));
        }
    }
#undef CKS
    return SOBEK_OK;
}
