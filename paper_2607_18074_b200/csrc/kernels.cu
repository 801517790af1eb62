// Device kernels of the streaming convolution (sm_100a).
//
//   k_pack_R<UNPACK>      : the accumulated R adjoint, kept per group as gRp_g[(pi,u,q), w],
//                           back into the layout of R[K, N_w]
// (the edge stream lives in edge_stream*.cu, the receiver-owned edge pass in edge_pass.cu, the
//  node-side contractions in gemm_tc.cu)

#include <algorithm>
#include <atomic>
#include <type_traits>
#include <vector>

#include "internal.h"

namespace sobek {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Optional per-kernel-class timing (off by default): every launch is bracketed by two CUDA
// events on the launching stream; sobek_timing_collect sums the elapsed times per class.
static bool g_timing = false;
struct TimedLaunch { cudaEvent_t a, b; int cls; };
static std::vector<TimedLaunch> g_timed;
static const char* kClassNames[K_NCLASS] = {"pack_R", "edge_stream_state", "node_gemm", "edge_pass", "fill", "fused_stream_gemm"};

KernelTimer::KernelTimer(int cls, cudaStream_t s) : cls_(cls), s_(s), on_(g_timing) {
    if (!on_) return;
    if (cudaEventCreate(&a_) != cudaSuccess || cudaEventCreate(&b_) != cudaSuccess) { on_ = false; return; }
    cudaEventRecord(a_, s_);
}
KernelTimer::~KernelTimer() {
    if (!on_) return;
    cudaEventRecord(b_, s_);
    g_timed.push_back(TimedLaunch{a_, b_, cls_});
}

Fork::Fork(const sobek_plan* p, cudaStream_t main) : p_(p), main_(main) {
    // while per-kernel timing is on, everything stays on the caller's stream so that the event
    // brackets of different kernels do not overlap
    if (p->n_side <= 0 || g_timing) return;
    if (cudaEventRecord(p->ev_fork, main) != cudaSuccess) { (void)cudaGetLastError(); return; }
    on_ = true;
}
cudaStream_t Fork::pick() {
    if (!on_) return main_;
    const int i = used_ % p_->n_side;
    if (used_ < p_->n_side) cudaStreamWaitEvent(p_->side[i], p_->ev_fork, 0);
    ++used_;
    return p_->side[i];
}
cudaError_t Fork::join() {
    if (!on_) return cudaSuccess;
    const int n = used_ < p_->n_side ? used_ : p_->n_side;
    for (int i = 0; i < n; ++i) {
        cudaError_t e = cudaEventRecord(p_->ev_join[i], p_->side[i]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(main_, p_->ev_join[i], 0);
        if (e != cudaSuccess) return e;
    }
    used_ = 0;
    on_ = false;
    return cudaSuccess;
}

}  // namespace sobek

extern "C" int64_t sobek_launch_count(void) { return sobek::g_launches.load(); }

extern "C" int sobek_timing_enable(int on) {
    sobek::g_timing = on != 0;
    return SOBEK_OK;
}

extern "C" int sobek_timing_classes(void) { return sobek::K_NCLASS; }

extern "C" const char* sobek_timing_class_name(int cls) {
    return (cls >= 0 && cls < sobek::K_NCLASS) ? sobek::kClassNames[cls] : "";
}

extern "C" int sobek_timing_collect(double* total_ms, int64_t* launches) {
    if (!total_ms || !launches) return SOBEK_ERR_INVALID_ARG;
    for (int c = 0; c < sobek::K_NCLASS; ++c) { total_ms[c] = 0.0; launches[c] = 0; }
    int rc = SOBEK_OK;
    for (auto& t : sobek::g_timed) {
        float ms = 0.f;
        if (cudaEventSynchronize(t.b) != cudaSuccess || cudaEventElapsedTime(&ms, t.a, t.b) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = SOBEK_ERR_CUDA;
        }
        total_ms[t.cls] += ms;
        launches[t.cls] += 1;
        cudaEventDestroy(t.a);
        cudaEventDestroy(t.b);
    }
    sobek::g_timed.clear();
    return rc;
}

namespace sobek {
namespace {

// ------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t owner_of_edge(const int64_t* __restrict__ row_ptr, int64_t N,
                                                 int64_t e) {
    // largest i with row_ptr[i] <= e   (rows may be empty)
    int64_t lo = 0, hi = N;   // invariant: row_ptr[lo] <= e < row_ptr[hi]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (__ldg(row_ptr + mid) <= e) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void k_fill_zero(float* __restrict__ p, int64_t n) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t st = (int64_t)gridDim.x * blockDim.x;
    for (; i < n; i += st) p[i] = 0.f;
}

// ------------------------------------------------------------------------------------
// R re-layout.  One blockIdx.y per path; element (us, q, n) of the path's slab:
//   forward    : us = u (input mult.), n = w      Rp[rp_off + (koff + q*c_in  + u)*c_out + w]
//   transposed : us = w (output mult.), n = u     Rt[rp_off + (koff + q*c_out + w)*c_in  + u]
// both read/write R[q*N_w + w_off + u*c_out + w].
// ------------------------------------------------------------------------------------
template <bool UNPACK>
__global__ void k_pack_R(const DPath* __restrict__ paths, int transposed, int K, int64_t N_w,
                         const float* __restrict__ src, float* __restrict__ dst) {
    const DPath P = paths[blockIdx.y];
    const int64_t total = (int64_t)K * P.c_src * P.c_dst;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i % P.c_dst);
        const int64_t r = i / P.c_dst;
        const int q = (int)(r % K);
        const int us = (int)(r / K);
        const int u = transposed ? n : us, w = transposed ? us : n;
        const int64_t ri = (int64_t)q * N_w + P.w_off + (int64_t)u * P.c_out + w;
        const int64_t pi = P.rp_off + ((int64_t)P.koff + (int64_t)q * P.c_src + us) * P.c_dst + n;
        if (UNPACK) dst[ri] = src[pi]; else dst[pi] = src[ri];
    }
}

}  // namespace

// ======================================================================================
// host launchers
// ======================================================================================
cudaError_t launch_fill_zero(float* p, int64_t n, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 8);
    KernelTimer kt(K_FILL, s);
    k_fill_zero<<<blocks, 256, 0, s>>>(p, n);
    count_launch();
    return cudaGetLastError();
}

namespace {
// one thread per element of the ir_mul side (block offset + m*c + u); the mul_ir partner is block offset + u*d + m
__global__ void k_relayout(const float* __restrict__ src, float* __restrict__ dst, int64_t N, int C,
                           const int4* __restrict__ blocks, int nblk, int to_ir_mul) {
    const int64_t total = N * C;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t n = i / C;
        const int col = (int)(i - n * C);
        int b = 0;
        while (b + 1 < nblk && blocks[b + 1].x <= col) ++b;
        const int4 B = blocks[b];
        const int r = col - B.x, m = r / B.y, u = r - m * B.y;      // ir_mul position inside the block
        const int64_t other = n * C + B.x + u * B.z + m;
        if (to_ir_mul) dst[i] = src[other];
        else dst[other] = src[i];
    }
}
}  // namespace

cudaError_t launch_relayout(const float* src, float* dst, int64_t N, int C, const int4* blocks, int nblk, int to_ir_mul,
                            cudaStream_t s) {
    if (N <= 0 || C <= 0) return cudaSuccess;
    const int nb = (int)std::min<int64_t>((N * C + 255) / 256, 148 * 16);
    KernelTimer kt(K_PACK, s);
    k_relayout<<<nb, 256, 0, s>>>(src, dst, N, C, blocks, nblk, to_ir_mul);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_unpack_R(const sobek_plan* p, const Direction& dir, const float* Rp, float* R,
                            cudaStream_t s) {
    dim3 grid(32, (unsigned)dir.paths.size());
    KernelTimer kt(K_PACK, s);
    k_pack_R<true><<<grid, 256, 0, s>>>(dir.d_paths, 0, p->K, p->N_w, Rp, R);
    count_launch();
    return cudaGetLastError();
}

}  // namespace sobek

// ---- FP32 multiply-add peak of the device, measured (instrumentation; the paper has no counterpart) ----------
// Every thread runs 16 independent fused multiply-add chains, so that the FP32 pipes never wait for a result:
// 2 x 16 x FMA_ITERS flops per thread.  The accumulators are stored at the end so that the loop is not removed.
namespace sobek {
namespace {
constexpr int FMA_ITERS = 1 << 14;
__global__ void __launch_bounds__(1024) k_fma_peak(float* out, float a, float b) {
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = (float)(threadIdx.x + i);
#pragma unroll 1
    for (int it = 0; it < FMA_ITERS; it += 4) {
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) s += acc[i];
    out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}
}  // namespace
}  // namespace sobek

extern "C" int sobek_measure_fp32_peak(double seconds, float* scratch, size_t scratch_floats, double* tflops, void* stream) {
    using namespace sobek;
    if (!tflops || !scratch || !(seconds > 0.0) || seconds > 10.0) return SOBEK_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return SOBEK_ERR_CUDA;
    }
    const int blocks = sms * 2 * 4, threads = 1024;     // 2 resident CTAs of 1024 threads per SM, four waves
    if (scratch_floats < (size_t)blocks * threads) return SOBEK_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { (void)cudaGetLastError(); return SOBEK_ERR_CUDA; }
    const double flops_per_launch = 2.0 * 16.0 * FMA_ITERS * (double)blocks * threads;
    double total_ms = 0.0, best = 0.0;
    int launches = 0;
    int rc = SOBEK_OK;
    k_fma_peak<<<blocks, threads, 0, s>>>(scratch, 1.0000001f, 1e-7f);     // warm-up
    while (total_ms < seconds * 1e3 && launches < 100000) {
        cudaEventRecord(e0, s);
        for (int r = 0; r < 8; ++r) k_fma_peak<<<blocks, threads, 0, s>>>(scratch, 1.0000001f, 1e-7f);
        cudaEventRecord(e1, s);
        if (cudaEventSynchronize(e1) != cudaSuccess) { rc = SOBEK_ERR_CUDA; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        count_launch(8);
        total_ms += ms; launches += 8;
        if (ms > 0.f) best = std::max(best, 8.0 * flops_per_launch / (ms * 1e-3) / 1e12);
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    if (cudaGetLastError() != cudaSuccess) rc = SOBEK_ERR_CUDA;
    // the sustained figure: all launches over all the time
    *tflops = total_ms > 0.0 ? launches * flops_per_launch / (total_ms * 1e-3) / 1e12 : 0.0;
    (void)best;
    return rc;
}
