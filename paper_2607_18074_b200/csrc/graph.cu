// Graph preparation: validation of the receiver-sorted CSR and construction of the stable
// sender-sorted view (src_ptr, src_perm).  Integer work only; the result is unique
// (edges of one sender appear in increasing edge id), so it does not depend on the order
// in which threads run even though the placement step uses integer atomics.
#include "guard.cuh"
#include "internal.h"

namespace sobek {
namespace {

// status bits written to ws[0]
constexpr int kBadRowPtr = 1, kBadCol = 2;

__global__ void k_validate_count(int64_t N, int64_t E, const int64_t* __restrict__ row_ptr,
                                 const int32_t* __restrict__ col, unsigned long long* __restrict__ cnt,
                                 int* __restrict__ status) {
    const int64_t st = (int64_t)gridDim.x * blockDim.x;
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    for (int64_t i = t; i < N; i += st)
        if (row_ptr[i] > row_ptr[i + 1] || row_ptr[i] < 0) atomicOr(status, kBadRowPtr);
    if (t == 0 && (row_ptr[0] != 0 || row_ptr[N] != E)) atomicOr(status, kBadRowPtr);
    for (int64_t e = t; e < E; e += st) {
        const int32_t c = col[e];
        if (c < 0 || c >= N) atomicOr(status, kBadCol);
        else atomicAdd(cnt + c, 1ull);
    }
}

// exclusive scan of cnt[0..N) into src_ptr[0..N], three phases
constexpr int SCAN_T = 256, SCAN_PER = 8, SCAN_BLOCK = SCAN_T * SCAN_PER;

__global__ void k_scan_block_sums(int64_t N, const unsigned long long* __restrict__ cnt,
                                  unsigned long long* __restrict__ bsum) {
    __shared__ unsigned long long sh[SCAN_T];
    const int64_t base = (int64_t)blockIdx.x * SCAN_BLOCK;
    unsigned long long s = 0;
    for (int k = 0; k < SCAN_PER; ++k) {
        const int64_t i = base + threadIdx.x * SCAN_PER + k;
        if (i < N) s += cnt[i];
    }
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int o = SCAN_T / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) bsum[blockIdx.x] = sh[0];
}

__global__ void k_scan_bsums(int64_t nb, unsigned long long* __restrict__ bsum) {
    // single thread: nb is N/2048, at most a few thousand
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        unsigned long long run = 0;
        for (int64_t i = 0; i < nb; ++i) { const unsigned long long v = bsum[i]; bsum[i] = run; run += v; }
    }
}

__global__ void k_scan_final(int64_t N, int64_t E, const unsigned long long* __restrict__ cnt,
                             const unsigned long long* __restrict__ bsum, int64_t* __restrict__ src_ptr,
                             unsigned long long* __restrict__ cursor) {
    __shared__ unsigned long long sh[SCAN_T];
    const int64_t base = (int64_t)blockIdx.x * SCAN_BLOCK;
    unsigned long long loc[SCAN_PER];
    unsigned long long s = 0;
    for (int k = 0; k < SCAN_PER; ++k) {
        const int64_t i = base + threadIdx.x * SCAN_PER + k;
        loc[k] = s;
        if (i < N) s += cnt[i];
    }
    sh[threadIdx.x] = s;
    __syncthreads();
    // inclusive Hillis-Steele over thread totals
    for (int o = 1; o < SCAN_T; o <<= 1) {
        unsigned long long v = 0;
        if (threadIdx.x >= o) v = sh[threadIdx.x - o];
        __syncthreads();
        sh[threadIdx.x] += v;
        __syncthreads();
    }
    const unsigned long long off = bsum[blockIdx.x] + (threadIdx.x ? sh[threadIdx.x - 1] : 0ull);
    for (int k = 0; k < SCAN_PER; ++k) {
        const int64_t i = base + threadIdx.x * SCAN_PER + k;
        if (i < N) { src_ptr[i] = (int64_t)(off + loc[k]); cursor[i] = off + loc[k]; }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) src_ptr[N] = E;
}

__global__ void k_place(int64_t E, const int32_t* __restrict__ col, unsigned long long* __restrict__ cursor,
                        int32_t* __restrict__ tmp) {
    const int64_t st = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < E; e += st) {
        const unsigned long long pos = atomicAdd(cursor + col[e], 1ull);
        tmp[pos] = (int32_t)e;
    }
}

// one warp per sender segment: rank every edge id among the segment's ids and write it to
// its rank => increasing edge id inside the segment, whatever order k_place produced.
__global__ void k_sort_segments(int64_t N, const int64_t* __restrict__ src_ptr,
                                const int32_t* __restrict__ tmp, int32_t* __restrict__ perm) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t j = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5; j < N; j += warps) {
        const int64_t s0 = src_ptr[j], s1 = src_ptr[j + 1];
        for (int64_t a = s0 + lane; a < s1; a += 32) {
            const int32_t v = tmp[a];
            int64_t rank = 0;
            for (int64_t b = s0; b < s1; ++b) rank += (tmp[b] < v);
            perm[s0 + rank] = v;
        }
    }
}

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace

size_t graph_prepare_bytes(int64_t N, int64_t E) {
    const int64_t nb = (N + SCAN_BLOCK - 1) / SCAN_BLOCK + 1;
    return kHeaderBytes + align256((size_t)(N + 1) * 8) * 2 + align256((size_t)nb * 8) +
           align256((size_t)std::max<int64_t>(E, 1) * 4);
}

int graph_prepare(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* col, int64_t* src_ptr,
                  int32_t* src_perm, void* ws, size_t ws_bytes, cudaStream_t s) {
    if (N < 0 || E < 0 || !row_ptr || (!col && E > 0) || !src_ptr || (!src_perm && E > 0)) return SOBEK_ERR_INVALID_ARG;
    if (N >= (int64_t(1) << 31) || E >= (int64_t(1) << 31)) return SOBEK_ERR_UNSUPPORTED;   // int32 ids
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < graph_prepare_bytes(N, E)) return SOBEK_ERR_WORKSPACE;
    char* w = (char*)ws;
    int* status = (int*)w;
    w += kHeaderBytes;
    unsigned long long* cnt = (unsigned long long*)w; w += align256((size_t)(N + 1) * 8);
    unsigned long long* cursor = (unsigned long long*)w; w += align256((size_t)(N + 1) * 8);
    const int64_t nb = (N + SCAN_BLOCK - 1) / SCAN_BLOCK;
    unsigned long long* bsum = (unsigned long long*)w; w += align256((size_t)(nb + 1) * 8);
    int32_t* tmp = (int32_t*)w;
    cudaError_t e = cudaMemsetAsync(ws, 0, kHeaderBytes + align256((size_t)(N + 1) * 8), s);
    if (e != cudaSuccess) return SOBEK_ERR_CUDA;
    if (N == 0) {
        // only src_ptr[0] = 0 to write
        e = cudaMemsetAsync(src_ptr, 0, 8, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        return e == cudaSuccess ? (E == 0 ? SOBEK_OK : SOBEK_ERR_GRAPH) : SOBEK_ERR_CUDA;
    }
    const int T = 256;
    const int gridE = (int)std::min<int64_t>((std::max(E, N) + T - 1) / T, 148 * 16);
    k_validate_count<<<gridE, T, 0, s>>>(N, E, row_ptr, col, cnt, status);
    k_scan_block_sums<<<(unsigned)nb, SCAN_T, 0, s>>>(N, cnt, bsum);
    k_scan_bsums<<<1, 32, 0, s>>>(nb, bsum);
    k_scan_final<<<(unsigned)nb, SCAN_T, 0, s>>>(N, E, cnt, bsum, src_ptr, cursor);
    count_launch(4);
    int hstatus = 0;
    e = cudaMemcpyAsync(&hstatus, status, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return SOBEK_ERR_CUDA; }
    if (hstatus) return SOBEK_ERR_GRAPH;    // do not place edges whose sender is out of range
    if (E > 0) {
        k_place<<<gridE, T, 0, s>>>(E, col, cursor, tmp);
        const int gridS = (int)std::min<int64_t>((N * 32 + T - 1) / T, 148 * 16);
        k_sort_segments<<<gridS, T, 0, s>>>(N, src_ptr, tmp, src_perm);
        count_launch(2);
    }
    e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { (void)cudaGetLastError(); return SOBEK_ERR_CUDA; }
    return SOBEK_OK;
}

namespace {
// src_recv[p] = receiver of edge src_perm[p]: the row of the receiver CSR that holds that edge id
__global__ void k_receivers(int64_t N, int64_t E, const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ src_perm,
                            int32_t* __restrict__ src_recv) {
    for (int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; p < E; p += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = src_perm[p];
        int64_t lo = 0, hi = N;   // row_ptr[lo] <= e < row_ptr[hi]
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (row_ptr[mid] <= e) lo = mid; else hi = mid;
        }
        src_recv[p] = (int32_t)lo;
    }
}
}  // namespace

int graph_receivers(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* src_perm, int32_t* src_recv,
                    cudaStream_t s) {
    if (N < 0 || E < 0 || (E > 0 && (N == 0 || !row_ptr || !src_perm || !src_recv))) return SOBEK_ERR_INVALID_ARG;
    if (E == 0) return SOBEK_OK;
    const int grid = (int)std::min<int64_t>((E + 255) / 256, 148 * 16);
    k_receivers<<<grid, 256, 0, s>>>(N, E, row_ptr, src_perm, src_recv);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return SOBEK_ERR_CUDA;
    return SOBEK_OK;
}

namespace {
// rvec[e] = pos[sender(e)] - pos[receiver(e)]: one warp per receiver walks its edge segment
__global__ void k_edge_vectors(int64_t N, int64_t E, const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                               const float* __restrict__ pos, float* __restrict__ rvec) {
    const int lane = threadIdx.x & 31;
    const int64_t w0 = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5, nw = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t n = w0; n < N; n += nw) {
        const int64_t s0 = max((int64_t)0, min(row_ptr[n], E)), s1 = max(s0, min(row_ptr[n + 1], E));
        const float px = pos[3 * n], py = pos[3 * n + 1], pz = pos[3 * n + 2];
        for (int64_t e = s0 + lane; e < s1; e += 32) {
            const int64_t j = col[e];
            const bool ok = j >= 0 && j < N;      // an id out of range leaves a unit vector (and shows up in the conv calls)
            rvec[3 * e] = ok ? pos[3 * j] - px : 0.f;
            rvec[3 * e + 1] = ok ? pos[3 * j + 1] - py : 0.f;
            rvec[3 * e + 2] = ok ? pos[3 * j + 2] - pz : 1.f;
        }
    }
}
// gpos[n] = sum over the edges n sends (sender view, in its order) - sum over the edges n receives (in edge order):
// one thread per node, so that every sum has a fixed order
__global__ void k_position_gradient(int64_t N, int64_t E, const int64_t* __restrict__ row_ptr, const int64_t* __restrict__ src_ptr,
                                    const int32_t* __restrict__ src_perm, const float* __restrict__ g, float* __restrict__ gpos) {
    for (int64_t n = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; n < N; n += (int64_t)gridDim.x * blockDim.x) {
        float ax = 0.f, ay = 0.f, az = 0.f;
        const int64_t p0 = max((int64_t)0, min(src_ptr[n], E)), p1 = max(p0, min(src_ptr[n + 1], E));
        for (int64_t p = p0; p < p1; ++p) {
            const int64_t e = src_perm[p];
            if (e >= 0 && e < E) { ax += g[3 * e]; ay += g[3 * e + 1]; az += g[3 * e + 2]; }
        }
        const int64_t s0 = max((int64_t)0, min(row_ptr[n], E)), s1 = max(s0, min(row_ptr[n + 1], E));
        for (int64_t e = s0; e < s1; ++e) { ax -= g[3 * e]; ay -= g[3 * e + 1]; az -= g[3 * e + 2]; }
        gpos[3 * n] = ax; gpos[3 * n + 1] = ay; gpos[3 * n + 2] = az;
    }
}
}  // namespace

int edge_vectors(const sobek_graph* g, const float* pos, float* rvec, cudaStream_t s) {
    if (!g || g->N < 0 || g->E < 0 || (g->E > 0 && (!g->row_ptr || !g->col || !pos || !rvec))) return SOBEK_ERR_INVALID_ARG;
    if (g->E == 0) return SOBEK_OK;
    const int grid = (int)std::min<int64_t>((g->N + 7) / 8, 148 * 16);
    k_edge_vectors<<<grid, 256, 0, s>>>(g->N, g->E, g->row_ptr, g->col, pos, rvec);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SOBEK_OK : SOBEK_ERR_CUDA;
}

int position_gradient(const sobek_graph* g, const float* g_rvec, float* gpos, cudaStream_t s) {
    if (!g || g->N < 0 || g->E < 0 || (g->N > 0 && !gpos) || (g->E > 0 && (!g->row_ptr || !g_rvec))) return SOBEK_ERR_INVALID_ARG;
    if (g->E > 0 && (!g->src_ptr || !g->src_perm)) return SOBEK_ERR_NEED_TRANSPOSE;
    if (g->N == 0) return SOBEK_OK;
    if (g->E == 0) return cudaMemsetAsync(gpos, 0, (size_t)g->N * 12, s) == cudaSuccess ? SOBEK_OK : SOBEK_ERR_CUDA;
    const int grid = (int)std::min<int64_t>((g->N + 127) / 128, 148 * 16);
    k_position_gradient<<<grid, 128, 0, s>>>(g->N, g->E, g->row_ptr, g->src_ptr, g->src_perm, g_rvec, gpos);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SOBEK_OK : SOBEK_ERR_CUDA;
}

// ---- processing order of the nodes of a chunk (load balance of the persistent edge kernels) -------------------------
namespace {
constexpr int ORD_BINS = 2048;
__global__ void __launch_bounds__(1024) k_chunk_order(const int64_t* __restrict__ ptr, int64_t N, int64_t E, int64_t chunk,
                                                      int period, int4* __restrict__ oseg, int* status) {
    __shared__ int hist[ORD_BINS];
    __shared__ int wsum[32];
    const int64_t n0 = (int64_t)blockIdx.x * chunk;
    const int64_t nn = min(chunk, N - n0);
    for (int i = threadIdx.x; i < ORD_BINS; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    // bucket = ORD_BINS - 1 - min(length, ORD_BINS - 1): longest segments first
    for (int64_t i = threadIdx.x; i < nn; i += blockDim.x) {
        int64_t s0, s1;
        seg_bounds(ptr, n0 + i, E, status, s0, s1);
        atomicAdd(&hist[ORD_BINS - 1 - (int)min(s1 - s0, (int64_t)(ORD_BINS - 1))], 1);
    }
    __syncthreads();
    // exclusive scan of the histogram: two bins per thread, warp scans, then the warp totals
    {
        const int t = threadIdx.x, lane = t & 31, w = t >> 5;
        const int a0 = hist[2 * t], a1 = hist[2 * t + 1];
        int v = a0 + a1;
        for (int d = 1; d < 32; d <<= 1) { const int u = __shfl_up_sync(0xffffffffu, v, d); if (lane >= d) v += u; }
        if (lane == 31) wsum[w] = v;
        __syncthreads();
        if (w == 0) {
            int x = wsum[lane];
            for (int d = 1; d < 32; d <<= 1) { const int u = __shfl_up_sync(0xffffffffu, x, d); if (lane >= d) x += u; }
            wsum[lane] = x;
        }
        __syncthreads();
        const int base = (w > 0 ? wsum[w - 1] : 0) + v - (a0 + a1);
        hist[2 * t] = base;
        hist[2 * t + 1] = base + a0;
    }
    __syncthreads();
    const int64_t full = (nn / period) * period;       // entries in whole rounds
    for (int64_t i = threadIdx.x; i < nn; i += blockDim.x) {
        int64_t s0, s1;
        seg_bounds(ptr, n0 + i, E, nullptr, s0, s1);
        const int64_t r = atomicAdd(&hist[ORD_BINS - 1 - (int)min(s1 - s0, (int64_t)(ORD_BINS - 1))], 1);
        int64_t v = r;
        if (r < full) {                                  // every second whole round runs backwards
            const int64_t round = r / period, k = r - round * period;
            if (round & 1) v = round * period + (period - 1 - k);
        }
        oseg[n0 + v] = make_int4((int)i, (int)s0, (int)s1, 0);
    }
}
}  // namespace

cudaError_t launch_chunk_order(const EdgeView& ev, int64_t chunk, int period, int4* oseg, int* status, cudaStream_t s) {
    if (ev.N <= 0 || chunk <= 0 || !oseg) return cudaSuccess;
    const int64_t n_chunks = (ev.N + chunk - 1) / chunk;
    k_chunk_order<<<(unsigned)n_chunks, 1024, 0, s>>>(ev.ptr, ev.N, ev.E, chunk, period, oseg, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace sobek
