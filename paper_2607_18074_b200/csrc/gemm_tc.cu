// Node-side contractions on the 5th-generation tensor cores (tcgen05, accumulators in TMEM,
// operands staged by TMA).
//
// fp32 parity on bf16 tensor cores: every fp32 operand a is split as a = a_hi + a_lo with
// a_hi = bf16(a), a_lo = bf16(a - a_hi), and a product is evaluated in three passes
//     a*b ~= a_hi*b_hi + a_lo*b_hi + a_hi*b_lo        (fp32 accumulation in TMEM)
// which leaves a relative error of about 2^-16 per product (the dropped a_lo*b_lo term and the
// second-order remainders), well inside the 1e-4 / 5e-4 max-norm tolerances.
//
// Kernel k_gemm_tc computes  C[M,N] (+)= A[M,Kd] * B[N,Kd]^T  for row-major ("K-major") bf16
// operands (hi and lo parts), used for
//     y   = Z  * Rp          (Eq. receiver_matrix_product;  A = Z,  B = Rp^T  [w][k])
//     Zbar = gy * Rp^T       (Eq. receiver_adjoint;         A = gy, B = Rp    [k][w])
// and, with MN-major operand descriptors (TRANSPOSED_AB), for the weight adjoint
//     gRp = Z^T * gy         (Eq. receiver_adjoint;  A^T = Z [r][k],  B^T = gy [r][w]).
//
// CTA = 192 threads: warp 0 issues TMA loads, warp 1 allocates TMEM and issues tcgen05.mma,
// warps 2..5 drain the accumulator (tcgen05.ld) and write C.  Every mbarrier wait is bounded:
// if it gives up it records SOBEK_ERR_DEVICE_TIMEOUT in the status word and carries on, so the
// kernel always reaches its TMEM release and returns.
#include <cuda_bf16.h>

#include <algorithm>
#include <new>

#include "internal.h"
#include "ptx.cuh"

namespace sobek {
namespace {

using namespace ptx;

constexpr int BM = 128;     // rows of C per CTA (UMMA M)
constexpr int BK = 64;      // bf16 elements per k-block = one 128-byte swizzle row
constexpr int TC_THREADS = 192;

struct TcArgs {
    float* C;
    __nv_bfloat16* Ch;          // when set, the result is written as bf16 (hi, lo) at the same indices instead of C
    __nv_bfloat16* Cl;
    int64_t c_outer, c_inner;   // C(m,n) = C[(m/c_d)*c_outer + (m%c_d)*c_inner + n]
    int32_t c_d;
    int32_t accumulate;
    int32_t passes;             // 3: split-bf16 product (fp32-faithful); 1: the hi x hi product only (plain bf16 GEMM)
    int64_t M, N, Kd;
    int32_t BN;                 // tile width (multiple of 16, <= 256)
    int32_t stages;
    int32_t ring_bytes;         // bytes of the operand ring = what the epilogue may use as its staging area
    int32_t tmem_cols;          // power of two >= max(32, BN)
    int32_t mn_major;           // 0: A[M,Kd], B[N,Kd] row-major;  1: A^T[Kd,M], B^T[Kd,N] row-major
    int32_t splits;             // gridDim.z: the contraction range is cut into this many pieces,
    int64_t split_stride;       //   piece z writes its partial result to C + z*split_stride
    int* status;
};

// One launch runs up to TC_MAX_BATCH independent products (the output groups of one node-side step): the CTAs
// tile0[b] .. tile0[b+1]-1 belong to product b and number its (m tile, n tile, split) triples.
constexpr int TC_MAX_BATCH = 5;
constexpr unsigned kSmallQueueTiles = 592;     // two CTAs on each of 148 SMs, twice over
struct alignas(64) TcProblem {
    CUtensorMap tmAh, tmAl, tmBh, tmBl;
    TcArgs g;
    uint32_t gx, gy;            // m tiles, n tiles
};
struct TcBatch {
    TcProblem p[TC_MAX_BATCH];
    int32_t n;
    uint32_t tile0[TC_MAX_BATCH + 1];
};
static_assert(sizeof(TcBatch) <= sizeof(GemmBatch::storage), "GemmBatch::storage holds a TcBatch");

__global__ void __launch_bounds__(TC_THREADS, 2)
k_gemm_tc(const __grid_constant__ TcBatch B) {
    int bi = 0;
    while (bi + 1 < B.n && blockIdx.x >= B.tile0[bi + 1]) ++bi;
    const TcProblem& pr = B.p[bi];
    const TcArgs g = pr.g;        // by value: read once (the product is picked by a run-time index into the parameter)
    const CUtensorMap& tmAh = pr.tmAh;
    const CUtensorMap& tmAl = pr.tmAl;
    const CUtensorMap& tmBh = pr.tmBh;
    const CUtensorMap& tmBl = pr.tmBl;
    const uint32_t tile = blockIdx.x - B.tile0[bi];
    const uint32_t bx = tile % pr.gx, by = (tile / pr.gx) % pr.gy, bz = tile / (pr.gx * pr.gy);
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the 128-byte swizzle atoms
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_bytes = BM * BK * 2;             // 16 KiB
    const uint32_t b_bytes = (uint32_t)g.BN * BK * 2;
    const uint32_t stage_bytes = 2 * a_bytes + 2 * b_bytes;
    uint64_t* bars = (uint64_t*)(smem + (size_t)g.ring_bytes);
    // bars[0..S) full, bars[S..2S) empty, bars[2S] accumulator ready; then the TMEM base word
    uint32_t* tmem_holder = (uint32_t*)(bars + 2 * g.stages + 1);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = smem_u32(bars);
    const int S = g.stages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = (int)bx * BM, n0 = (int)by * g.BN;
    const int num_kb_all = (int)((g.Kd + BK - 1) / BK);
    const int kb_per = (num_kb_all + g.splits - 1) / g.splits;
    const int kb_first = (int)bz * kb_per;
    const int num_kb = max(0, min(kb_per, num_kb_all - kb_first));   // k-blocks of this piece

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(bar0 + 8 * s, 1); mbar_init(bar0 + 8 * (S + s), 1); }
        mbar_init(bar0 + 8 * 2 * S, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % S;
                const uint32_t ph = (kb / S) & 1;
                mbar_wait(bar0 + 8 * (S + s), ph ^ 1, g.status);        // slot free
                const uint32_t full = bar0 + 8 * s;
                mbar_expect_tx(full, g.passes == 1 ? a_bytes + b_bytes : stage_bytes);
                const uint32_t sa = sbase + s * stage_bytes;
                if (!g.mn_major) {
                    tma_load_2d(sa, &tmAh, (kb_first + kb) * BK, m0, full);
                    tma_load_2d(sa + 2 * a_bytes, &tmBh, (kb_first + kb) * BK, n0, full);
                    if (g.passes != 1) {
                        tma_load_2d(sa + a_bytes, &tmAl, (kb_first + kb) * BK, m0, full);
                        tma_load_2d(sa + 2 * a_bytes + b_bytes, &tmBl, (kb_first + kb) * BK, n0, full);
                    }
                } else {
                    // operands stored [Kd rows][M or N contiguous]: boxes of 64 MN-elements x 64 k-rows
                    for (int j = 0; j < BM / 64; ++j) {
                        tma_load_2d(sa + j * (64 * BK * 2), &tmAh, m0 + 64 * j, (kb_first + kb) * BK, full);
                        if (g.passes != 1) tma_load_2d(sa + a_bytes + j * (64 * BK * 2), &tmAl, m0 + 64 * j, (kb_first + kb) * BK, full);
                    }
                    for (int j = 0; j < g.BN / 64; ++j) {
                        tma_load_2d(sa + 2 * a_bytes + j * (64 * BK * 2), &tmBh, n0 + 64 * j, (kb_first + kb) * BK, full);
                        if (g.passes != 1) tma_load_2d(sa + 2 * a_bytes + b_bytes + j * (64 * BK * 2), &tmBl, n0 + 64 * j, (kb_first + kb) * BK, full);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: D = F32, A = B = BF16, M = 128, N = BN
            uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(g.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            if (g.mn_major) idesc |= (1u << 15) | (1u << 16);
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % S;
                const uint32_t ph = (kb / S) & 1;
                mbar_wait(bar0 + 8 * s, ph, g.status);                  // operands landed
                tc_fence_after();
                const uint32_t sa = sbase + s * stage_bytes;
                const uint32_t ah = sa, al = sa + a_bytes, bh = sa + 2 * a_bytes, bl = bh + b_bytes;
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                    uint64_t dAh, dAl, dBh, dBl;
                    if (!g.mn_major) {
                        // K-major: rows of 128 B, 8-row groups 1024 B apart; 16 k-elements = 32 B
                        dAh = make_desc(ah + 32 * k, 16, 1024); dAl = make_desc(al + 32 * k, 16, 1024);
                        dBh = make_desc(bh + 32 * k, 16, 1024); dBl = make_desc(bl + 32 * k, 16, 1024);
                    } else {
                        // MN-major: 64 MN-elements per 128-B row, 8 k-rows per 1024-B group (stride),
                        // next 64 MN-elements one box further (leading); 16 k = two groups
                        dAh = make_desc(ah + 2048 * k, 64 * BK * 2, 1024); dAl = make_desc(al + 2048 * k, 64 * BK * 2, 1024);
                        dBh = make_desc(bh + 2048 * k, 64 * BK * 2, 1024); dBl = make_desc(bl + 2048 * k, 64 * BK * 2, 1024);
                    }
                    const uint32_t first = (kb > 0 || k > 0) ? 1u : 0u;
                    tc_mma_bf16(tmem_base, dAh, dBh, idesc, first);
                    if (g.passes != 1) {
                        tc_mma_bf16(tmem_base, dAl, dBh, idesc, 1u);
                        tc_mma_bf16(tmem_base, dAh, dBl, idesc, 1u);
                    }
                }
                tc_commit(bar0 + 8 * (S + s));                           // frees the slot when the MMAs retire
            }
            tc_commit(bar0 + 8 * 2 * S);                                 // accumulator complete
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
        const int q = warp & 3;
        mbar_wait(bar0 + 8 * 2 * S, 0, g.status);
        tc_fence_after();
        // The pipeline buffers are idle now: each warp parks its 32 x BN block there and then writes C row by row
        // with the lanes along the columns (coalesced).
        if (g.Ch && (g.N & 7) == 0) {
            // bf16 (hi, lo) output.  The warp parks its 32 x BN block with a row pitch of BN + 4 floats (16-byte
            // pieces, conflict-free), then writes two rows per step: lanes 0-15 and 16-31 each convert 8 consecutive
            // columns of their row into two 16-byte stores, so that a row leaves as contiguous 256-byte runs.
            const int P4 = g.BN + 4;
            float* pk = reinterpret_cast<float*>(smem) + (size_t)q * 32 * P4;
            for (int c0 = 0; c0 < g.BN; c0 += 16) {
                float v[16];
                tc_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);   // warp-collective
#pragma unroll
                for (int j = 0; j < 16; j += 4)
                    *reinterpret_cast<float4*>(pk + lane * P4 + c0 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            }
            __syncwarp();
            const int half = lane >> 4, l16 = lane & 15;
            for (int r = half; r < 32; r += 2) {
                const int64_t m = (int64_t)m0 + q * 32 + r;
                if (m >= g.M) continue;
                const int64_t rbase = (int64_t)bz * g.split_stride + (int64_t)((uint32_t)m / (uint32_t)g.c_d) * g.c_outer + (int64_t)((uint32_t)m % (uint32_t)g.c_d) * g.c_inner;
                for (int c8 = l16; c8 < g.BN / 8; c8 += 16) {
                    const int64_t n = (int64_t)n0 + 8 * c8;
                    if (n < g.N) {
                        const float4 x0 = *reinterpret_cast<const float4*>(pk + r * P4 + 8 * c8);
                        const float4 x1 = *reinterpret_cast<const float4*>(pk + r * P4 + 8 * c8 + 4);
                        const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                        uint32_t hw[4], lw[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float a0 = num_kb > 0 ? xv[2 * j] : 0.f, a1 = num_kb > 0 ? xv[2 * j + 1] : 0.f;
                            const __nv_bfloat162 hp = __floats2bfloat162_rn(a0, a1);
                            const float2 hf = __bfloat1622float2(hp);
                            const __nv_bfloat162 lp = __floats2bfloat162_rn(a0 - hf.x, a1 - hf.y);
                            hw[j] = *reinterpret_cast<const uint32_t*>(&hp);
                            lw[j] = *reinterpret_cast<const uint32_t*>(&lp);
                        }
                        *reinterpret_cast<uint4*>(g.Ch + rbase + n) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        *reinterpret_cast<uint4*>(g.Cl + rbase + n) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    }
                }
            }
        } else {
        const int P4 = g.BN + 4;      // 16-byte-aligned pitch: conflict-free 16-byte writes, conflict-free row reads
        float* park = reinterpret_cast<float*>(smem) + (size_t)q * 32 * P4;
        for (int c0 = 0; c0 < g.BN; c0 += 16) {
            float v[16];
            tc_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);   // warp-collective
#pragma unroll
            for (int j = 0; j < 16; j += 4)
                *reinterpret_cast<float4*>(park + lane * P4 + c0 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
        __syncwarp();
        for (int r = 0; r < 32; ++r) {
            const int64_t m = (int64_t)m0 + q * 32 + r;
            if (m >= g.M) break;
            const int64_t rbase = (int64_t)bz * g.split_stride + (int64_t)((uint32_t)m / (uint32_t)g.c_d) * g.c_outer + (int64_t)((uint32_t)m % (uint32_t)g.c_d) * g.c_inner;
            float* crow = g.C + rbase;
            for (int c = lane; c < g.BN; c += 32) {
                const int64_t n = (int64_t)n0 + c;
                if (n < g.N) {
                    const float v = num_kb > 0 ? park[r * P4 + c] : 0.f;
                    if (g.Ch) {
                        const __nv_bfloat16 h = __float2bfloat16_rn(v);
                        g.Ch[rbase + n] = h;
                        g.Cl[rbase + n] = __float2bfloat16_rn(v - __bfloat162float(h));
                    } else {
                        crow[n] = g.accumulate ? crow[n] + v : v;
                    }
                }
            }
        }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------
// fp32 -> (bf16 hi, bf16 lo) with mapped source rows: dst[r*ld + c] for r < rows, c < cols
// ------------------------------------------------------------------------------------
__global__ void k_split(const float* __restrict__ src, int64_t s_outer, int64_t s_inner, int s_d,
                        int64_t rows, int cols, int64_t ld, __nv_bfloat16* __restrict__ hi,
                        __nv_bfloat16* __restrict__ lo) {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cols;
        const int c = (int)(i - r * cols);
        const float v = src[(r / s_d) * s_outer + (r % s_d) * s_inner + c];
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[r * ld + c] = h;
        lo[r * ld + c] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

// several such packings (directions, layouts, R or its direction vR) in one launch: blockIdx.z picks the job
struct PackJobsArg { PackJob j[kMaxPackJobs]; int K; int64_t N_w; };
__global__ void k_pack_R_jobs(const PackJobsArg J) {
    const PackJob q = J.j[blockIdx.z];
    if ((int)blockIdx.y >= q.n_paths) return;
    const DPath P = q.paths[blockIdx.y];
    const int gi = q.path_group[blockIdx.y];
    const int64_t base = q.grp_off[gi];
    const int64_t ld = q.grp_ld[gi];
    const int K = J.K;
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(q.hi);
    __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(q.lo);
    const int64_t total = (int64_t)K * P.c_src * P.c_dst;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i % P.c_dst);
        const int64_t r = i / P.c_dst;
        const int k1 = (int)(r % K);
        const int us = (int)(r / K);
        const int u = q.transposed ? n : us, w = q.transposed ? us : n;
        const float v = q.R[(int64_t)k1 * J.N_w + P.w_off + (int64_t)u * P.c_out + w];
        const int64_t k = (int64_t)P.koff + (int64_t)k1 * P.c_src + us;
        const int64_t o = q.n_major ? base + (int64_t)n * ld + k : base + k * ld + n;
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[o] = h;
        lo[o] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

// the same for several (source, destination) pairs in one launch: blockIdx.y picks the job
struct SplitJobs { SplitJob j[kMaxSplitJobs]; };
__global__ void k_split_jobs(const SplitJobs J) {
    const SplitJob q = J.j[blockIdx.y];
    const int64_t total = q.rows * q.cols;
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(q.hi);
    __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(q.lo);
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / q.cols;
        const int c = (int)(i - r * q.cols);
        const float v = q.src[(r / q.s_d) * q.s_outer + (r % q.s_d) * q.s_inner + c];
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[r * q.ld + c] = h;
        lo[r * q.ld + c] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

// R[K, N_w] -> bf16 hi/lo GEMM operands of one direction, per group g:
//   layout KN (n_major = 0): [k][c_dst] rows of length ldn_g      (B operand of Zbar = gy Rp^T)
//   layout NK (n_major = 1): [c_dst][k] rows of length ldk_g      (B operand of y = Z Rp)
__global__ void k_pack_R_bf16(const DPath* __restrict__ paths, const int64_t* __restrict__ grp_off,
                              const int32_t* __restrict__ grp_ld, const int32_t* __restrict__ path_group,
                              int transposed, int n_major, int K, int64_t N_w, const float* __restrict__ R,
                              __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
    const DPath P = paths[blockIdx.y];
    const int gi = path_group[blockIdx.y];
    const int64_t base = grp_off[gi];
    const int64_t ld = grp_ld[gi];
    const int64_t total = (int64_t)K * P.c_src * P.c_dst;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i % P.c_dst);
        const int64_t r = i / P.c_dst;
        const int q = (int)(r % K);
        const int us = (int)(r / K);
        const int u = transposed ? n : us, w = transposed ? us : n;
        const float v = R[(int64_t)q * N_w + P.w_off + (int64_t)u * P.c_out + w];
        const int64_t k = (int64_t)P.koff + (int64_t)q * P.c_src + us;
        const int64_t o = n_major ? base + (int64_t)n * ld + k : base + k * ld + n;
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[o] = h;
        lo[o] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

}  // namespace

int64_t round8(int64_t v) { return (v + 7) & ~int64_t(7); }

namespace {
// dst[i] += part[0][i] + part[1][i] + ... in this fixed order (deterministic split-K reduction)
__global__ void k_reduce_parts(float* __restrict__ dst, const float* __restrict__ part, int64_t n, int64_t stride,
                               int splits) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        float s = dst[i];
        for (int z = 0; z < splits; ++z) s += part[z * stride + i];
        dst[i] = s;
    }
}
struct ReduceRanges { ReduceRange r[kMaxReduceRanges]; };
__global__ void k_reduce_ranges(float* __restrict__ dst, const float* __restrict__ part, int64_t stride, const ReduceRanges R) {
    const ReduceRange rg = R.r[blockIdx.y];
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < rg.n; i += (int64_t)gridDim.x * blockDim.x) {
        float s = dst[rg.off + i];
        for (int z = 0; z < rg.splits; ++z) s += part[z * stride + rg.off + i];
        dst[rg.off + i] = s;
    }
}
}  // namespace

namespace {
// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever completes; the wait gives up after
// `limit_ns`, records SOBEK_ERR_DEVICE_TIMEOUT in the status word and the kernel returns normally.
__global__ void k_wait_selftest(int* status, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0, status, limit_ns);
    }
}
}  // namespace

cudaError_t launch_wait_selftest(int* status, uint64_t limit_ns, cudaStream_t s) {
    k_wait_selftest<<<1, 32, 0, s>>>(status, limit_ns);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_reduce_parts(float* dst, const float* part, int64_t n, int64_t stride, int splits, cudaStream_t s) {
    if (n <= 0 || splits <= 0) return cudaSuccess;
    const int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 8);
    KernelTimer kt(K_GEMM, s);
    k_reduce_parts<<<blocks, 256, 0, s>>>(dst, part, n, stride, splits);
    count_launch();
    return cudaGetLastError();
}

void PackQueue::add(const Direction& dir, int transposed, int n_major, const float* R, void* hi, void* lo) {
    if (p->uvu || n >= kMaxPackJobs) { overflow = overflow || (!p->uvu && n >= kMaxPackJobs); return; }
    j[n++] = PackJob{dir.d_paths, n_major ? dir.d_nk_off : dir.d_kn_off, n_major ? dir.d_nk_ld : dir.d_kn_ld, dir.d_path_group,
                     (int)dir.paths.size(), transposed, n_major, R, hi, lo};
}
cudaError_t PackQueue::flush(cudaStream_t s) {
    if (overflow) return cudaErrorInvalidValue;
    if (n == 0) return cudaSuccess;
    PackJobsArg J{};
    int max_paths = 0;
    for (int i = 0; i < n; ++i) { J.j[i] = j[i]; max_paths = std::max(max_paths, j[i].n_paths); }
    J.K = p->K; J.N_w = p->N_w;
    dim3 grid(32, (unsigned)max_paths, (unsigned)n);
    n = 0;
    if (max_paths == 0) return cudaSuccess;
    KernelTimer kt(K_PACK, s);
    k_pack_R_jobs<<<grid, 256, 0, s>>>(J);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_split_jobs(const SplitJob* jobs, int n, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    if (n > kMaxSplitJobs) return cudaErrorInvalidValue;
    SplitJobs J{};
    int64_t tmax = 0;
    for (int i = 0; i < n; ++i) { J.j[i] = jobs[i]; tmax = std::max(tmax, jobs[i].rows * jobs[i].cols); }
    if (tmax <= 0) return cudaSuccess;
    dim3 grid((unsigned)std::min<int64_t>((tmax + 255) / 256, 148 * 8), (unsigned)n);
    KernelTimer kt(K_PACK, s);
    k_split_jobs<<<grid, 256, 0, s>>>(J);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_reduce_ranges(float* dst, const float* part, int64_t stride, const ReduceRange* r, int nr, cudaStream_t s) {
    if (nr <= 0) return cudaSuccess;
    if (nr > kMaxReduceRanges) return cudaErrorInvalidValue;
    ReduceRanges R{};
    int64_t nmax = 0;
    for (int i = 0; i < nr; ++i) { R.r[i] = r[i]; nmax = std::max(nmax, r[i].n); }
    if (nmax <= 0) return cudaSuccess;
    dim3 grid((unsigned)std::min<int64_t>((nmax + 255) / 256, 148 * 4), (unsigned)nr);
    KernelTimer kt(K_GEMM, s);
    k_reduce_ranges<<<grid, 256, 0, s>>>(dst, part, stride, R);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_split(const float* src, int64_t s_outer, int64_t s_inner, int s_d, int64_t rows, int cols,
                         int64_t ld, void* hi, void* lo, cudaStream_t s) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    const int64_t total = rows * cols;
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, 148 * 16);
    KernelTimer kt(K_PACK, s);
    k_split<<<blocks, 256, 0, s>>>(src, s_outer, s_inner, s_d, rows, cols, ld, (__nv_bfloat16*)hi, (__nv_bfloat16*)lo);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_pack_R_bf16(const sobek_plan* p, const Direction& dir, int transposed, int n_major,
                               const float* R, void* hi, void* lo, cudaStream_t s) {
    dim3 grid(32, (unsigned)dir.paths.size());
    KernelTimer kt(K_PACK, s);
    k_pack_R_bf16<<<grid, 256, 0, s>>>(dir.d_paths, n_major ? dir.d_nk_off : dir.d_kn_off,
                                       n_major ? dir.d_nk_ld : dir.d_kn_ld, dir.d_path_group, transposed, n_major,
                                       p->K, p->N_w, R, (__nv_bfloat16*)hi, (__nv_bfloat16*)lo);
    count_launch();
    return cudaGetLastError();
}

// C[M,N] (+)= A * B^T on tensor cores.  mn_major = 0: A[M][lda], B[N][ldb] (rows contiguous in k).
// mn_major = 1: A^T[Kd][lda] (contiguous in m), B^T[Kd][ldb] (contiguous in n).
// gemm_tc_add queues one product (launching what is queued when the batch is full); gemm_tc_flush launches the queue.
cudaError_t gemm_tc_add(GemmBatch& gb, const void* Ahi, const void* Alo, int64_t lda, const void* Bhi, const void* Blo,
                        int64_t ldb, float* C, int64_t c_outer, int64_t c_inner, int c_d, int64_t M, int64_t N,
                        int64_t Kd, int accumulate, int mn_major, int* status, cudaStream_t s, int splits,
                        int64_t split_stride, void* Chi, void* Clo, int passes) {
    if (M <= 0 || N <= 0 || Kd <= 0) return cudaSuccess;
    if (M >= (int64_t(1) << 32)) return cudaErrorInvalidValue;   // the epilogue maps rows with 32-bit divisions
    TcBatch& B = *reinterpret_cast<TcBatch*>(gb.storage);
    TcProblem fresh;
    TcProblem& pr = fresh;
    TcArgs& g = pr.g;
    g = TcArgs{};
    g.C = C; g.Ch = (__nv_bfloat16*)Chi; g.Cl = (__nv_bfloat16*)Clo; g.c_outer = c_outer; g.c_inner = c_inner; g.c_d = c_d; g.accumulate = accumulate; g.passes = passes == 1 ? 1 : 3;
    g.M = M; g.N = N; g.Kd = Kd; g.mn_major = mn_major; g.status = status;
    g.splits = std::max(1, std::min<int>(splits, (int)((Kd + BK - 1) / BK))); g.split_stride = split_stride;
    int BN;
    const int num_kb = (int)((Kd + BK - 1) / BK);
    if (mn_major) BN = N <= 64 ? 64 : (N <= 128 ? 128 : 256);     // whole 64-wide boxes
    else BN = (int)std::min<int64_t>(num_kb <= 2 ? 128 : 256, (N + 15) / 16 * 16);   // one or two k-blocks are all epilogue: narrower tiles, more CTAs
    g.BN = BN;
    const size_t stage = 2 * (size_t)BM * BK * 2 + 2 * (size_t)BN * BK * 2;
    // two (or more) CTAs per SM where the ring fits twice (more loads and epilogues in flight per SM), else one
    // CTA with a deeper ring; never more stages than k-blocks
    int stages = (int)std::min<size_t>(4, (108 * 1024) / stage);
    if (stages < 2) stages = (int)std::min<size_t>(4, (200 * 1024) / stage);
    stages = std::max(1, std::min(stages, (num_kb + g.splits - 1) / g.splits));
    // one or two k-blocks per tile: the tile is all epilogue, and three CTAs per SM with a single stage each overlap
    // their epilogues better than one CTA with a stage per k-block
    if ((num_kb + g.splits - 1) / g.splits <= 2 && stage <= 72 * 1024) stages = 1;
    g.stages = stages;
    const size_t park = (size_t)4 * 32 * (BN + 4) * sizeof(float);       // epilogue staging of the four drain warps
    g.ring_bytes = (int32_t)((std::max(park, (size_t)stages * stage) + 1023) & ~size_t(1023));
    int cols = 32;
    while (cols < BN) cols <<= 1;
    g.tmem_cols = cols;
    bool ok;
    if (!mn_major) {
        ok = make_map(&pr.tmAh, Ahi, Kd, M, lda, BK, BM) && make_map(&pr.tmAl, Alo, Kd, M, lda, BK, BM) &&
             make_map(&pr.tmBh, Bhi, Kd, N, ldb, BK, BN) && make_map(&pr.tmBl, Blo, Kd, N, ldb, BK, BN);
    } else {
        ok = make_map(&pr.tmAh, Ahi, M, Kd, lda, 64, BK) && make_map(&pr.tmAl, Alo, M, Kd, lda, 64, BK) &&
             make_map(&pr.tmBh, Bhi, N, Kd, ldb, 64, BK) && make_map(&pr.tmBl, Blo, N, Kd, ldb, 64, BK);
    }
    if (!ok) return cudaErrorInvalidValue;
    pr.gx = (uint32_t)((M + BM - 1) / BM);
    pr.gy = (uint32_t)((N + BN - 1) / BN);
    const uint64_t tiles = (uint64_t)pr.gx * pr.gy * (uint64_t)g.splits;
    const size_t sh = (size_t)g.ring_bytes + 1024 + 8 * (2 * g.stages + 1) + 16;
    if (gb.n > 0 && (gb.n == TC_MAX_BATCH || tiles + B.tile0[gb.n] >= (uint64_t(1) << 31))) {
        cudaError_t e = gemm_tc_flush(gb, s, nullptr);
        if (e != cudaSuccess) return e;
    }
    if (tiles >= (uint64_t(1) << 31)) return cudaErrorInvalidValue;
    if (gb.n == 0) B.tile0[0] = 0;
    B.p[gb.n] = fresh;
    B.tile0[gb.n + 1] = B.tile0[gb.n] + (uint32_t)tiles;
    gb.sh = std::max(gb.sh, sh);
    gb.sh_of[gb.n] = sh;
    ++gb.n;
    return cudaSuccess;
}

namespace {
// one launch over the products q[0..n) of B (indices into B.p), in that order
void launch_sub(const TcBatch& B, const int* q, int n, size_t sh, cudaStream_t s) {
    TcBatch sub;
    sub.n = n;
    sub.tile0[0] = 0;
    for (int i = 0; i < n; ++i) {
        sub.p[i] = B.p[q[i]];
        sub.tile0[i + 1] = sub.tile0[i] + sub.p[i].gx * sub.p[i].gy * (uint32_t)sub.p[i].g.splits;
    }
    KernelTimer kt(K_GEMM, s);
    k_gemm_tc<<<sub.tile0[n], TC_THREADS, sh, s>>>(sub);
    count_launch();
}
}  // namespace

// One launch has one shared-memory size, the largest of its products, so a product that fits three CTAs on an SM runs
// one per SM beside a product that needs the whole SM (measured on the profile 128x0e + 64x1o + 64x2e:
// 30,872 single-k-block tiles took 1.57 ms in one launch with the 197 KB of the widest product against
// 0.75 ms in three launches).  Hence: a queue of at most kSmallQueueTiles tiles cannot fill the GPU anyway and runs as
// one launch (what counts there is the number of launches); a larger queue runs one launch per class of products with
// the same number of CTAs per SM, the classes side by side on the plan's side streams where a plan is given.
cudaError_t gemm_tc_flush(GemmBatch& gb, cudaStream_t s, const sobek_plan* p) {
    if (gb.n == 0) return cudaSuccess;
    TcBatch& B = *reinterpret_cast<TcBatch*>(gb.storage);
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    // longest contraction first: the CTAs that run longest start first, the short ones fill the tail
    int order[TC_MAX_BATCH];
    for (int i = 0; i < gb.n; ++i) order[i] = i;
    auto len = [&](int i) { return (B.p[i].g.Kd + B.p[i].g.splits - 1) / B.p[i].g.splits; };
    std::stable_sort(order, order + gb.n, [&](int x, int y) { return len(x) > len(y); });
    auto per_sm = [](size_t bytes) { return (int)std::min<size_t>(8, (size_t)(227 * 1024) / std::max<size_t>(bytes, 1)); };
    bool one_class = true;
    for (int i = 1; i < gb.n; ++i) one_class = one_class && per_sm(gb.sh_of[i]) == per_sm(gb.sh_of[0]);
    if (one_class || B.tile0[gb.n] <= kSmallQueueTiles) {
        launch_sub(B, order, gb.n, gb.sh, s);
    } else {
        bool done[TC_MAX_BATCH] = {};
        int n_class = 0;
        cudaError_t err = cudaSuccess;
        {
            // (a Fork only where there is a plan to take side streams from)
            Fork* fork = nullptr;
            alignas(Fork) unsigned char fork_mem[sizeof(Fork)];
            if (p) fork = new (fork_mem) Fork(p, s);
            for (int a = 0; a < gb.n; ++a) {
                const int ia = order[a];
                if (done[ia]) continue;
                int q[TC_MAX_BATCH], nq = 0;
                size_t sh = 0;
                for (int b = a; b < gb.n; ++b) {
                    const int ib = order[b];
                    if (!done[ib] && per_sm(gb.sh_of[ib]) == per_sm(gb.sh_of[ia])) { q[nq++] = ib; done[ib] = true; sh = std::max(sh, gb.sh_of[ib]); }
                }
                launch_sub(B, q, nq, sh, fork ? fork->pick() : s);
                ++n_class;
            }
            if (fork) { err = fork->join(); fork->~Fork(); }
        }
        if (err != cudaSuccess) return err;
    }
    gb.n = 0; gb.sh = 0;
    return cudaGetLastError();
}

cudaError_t launch_gemm_tc(const void* Ahi, const void* Alo, int64_t lda, const void* Bhi, const void* Blo,
                           int64_t ldb, float* C, int64_t c_outer, int64_t c_inner, int c_d, int64_t M, int64_t N,
                           int64_t Kd, int accumulate, int mn_major, int* status, cudaStream_t s, int splits,
                           int64_t split_stride, void* Chi, void* Clo, int passes) {
    GemmBatch gb;
    cudaError_t e = gemm_tc_add(gb, Ahi, Alo, lda, Bhi, Blo, ldb, C, c_outer, c_inner, c_d, M, N, Kd, accumulate, mn_major, status, s,
                                splits, split_stride, Chi, Clo, passes);
    if (e != cudaSuccess) return e;
    return gemm_tc_flush(gb, s, nullptr);
}

}  // namespace sobek
