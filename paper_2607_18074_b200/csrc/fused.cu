// Host side of the fused edge-stream + contraction kernels: stage lists, the stage-ordered bf16
// copy of R, and the launches (kernels in fused_impl.cuh, instantiated in fused_k*.cu).
#include <algorithm>

#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace sobek {

// Stages of one direction: for every group, every path, every block of 256/KP multiplicities (and, if
// K > 16, every chunk of 16 radial components).  The packed copy of R follows the same order with
// 256 columns per stage, zero where a stage is ragged.
void build_fused_stages(const sobek_plan* p, Direction& dir) {
    const int KP = p->K <= 8 ? 8 : 16;
    const int US = 256 / KP;
    dir.fstages.clear();
    dir.fs_begin.assign(dir.groups.size(), 0);
    dir.fs_count.assign(dir.groups.size(), 0);
    dir.fk_off.assign(dir.groups.size(), 0);
    dir.fk_elems = 0;
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        dir.fs_begin[gi] = (int)dir.fstages.size();
        for (int k = G.path_begin; k < G.path_end; ++k)
            for (int q0 = 0; q0 < p->K; q0 += KP)
                for (int u0 = 0; u0 < dir.paths[k].c_src; u0 += US) dir.fstages.push_back(FStage{k, u0, q0, (int)gi});
        dir.fs_count[gi] = (int)dir.fstages.size() - dir.fs_begin[gi];
        dir.fk_off[gi] = dir.fk_elems;
        dir.fk_elems += (int64_t)G.c_dst * dir.fs_count[gi] * 256;
    }
}

namespace {

__global__ void k_pack_R_fused(const DPath* __restrict__ paths, const FStage* __restrict__ stages,
                               const int64_t* __restrict__ fk_off, const int32_t* __restrict__ fs_begin,
                               const int32_t* __restrict__ fs_count, int transposed, int K, int KP, int64_t N_w,
                               const float* __restrict__ R, __nv_bfloat16* __restrict__ hi,
                               __nv_bfloat16* __restrict__ lo) {
    const int si = blockIdx.y;
    const FStage st = stages[si];
    const DPath P = paths[st.path];
    const int gi = st.group;
    const int sl = si - fs_begin[gi];
    const int64_t ld = (int64_t)fs_count[gi] * 256;
    const int US = 256 / KP;
    const int total = P.c_dst * 256;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int n = i >> 8, c = i & 255;
        const int ul = c / KP, q = c - ul * KP;
        const int us = st.u0 + ul;
        float v = 0.f;
        if (ul < US && us < P.c_src && st.q0 + q < K) {
            const int u = transposed ? n : us, w = transposed ? us : n;
            v = R[(int64_t)(st.q0 + q) * N_w + P.w_off + (int64_t)u * P.c_out + w];
        }
        const int64_t o = fk_off[gi] + (int64_t)n * ld + (int64_t)sl * 256 + c;
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[o] = h;
        lo[o] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

}  // namespace

bool fused_supported(const sobek_plan* p, const Direction& dir) {
    if (!p->use_fused) return false;
    for (const DGroup& G : dir.groups)
        if (G.path_end > G.path_begin && G.c_dst > 256) return false;
    return !dir.fstages.empty();
}

cudaError_t launch_pack_R_fused(const sobek_plan* p, const Direction& dir, int transposed, const float* R, void* hi,
                                void* lo, cudaStream_t s) {
    if (dir.fstages.empty()) return cudaSuccess;
    const int KP = p->K <= 8 ? 8 : 16;
    dim3 grid(32, (unsigned)dir.fstages.size());
    KernelTimer kt(K_PACK, s);
    k_pack_R_fused<<<grid, 256, 0, s>>>(dir.d_paths, dir.d_fstages, dir.d_fk_off, dir.d_fs_begin, dir.d_fs_count,
                                        transposed, p->K, KP, p->N_w, R, (__nv_bfloat16*)hi, (__nv_bfloat16*)lo);
    count_launch();
    return cudaGetLastError();
}

// dst (+)= (edge stream of the whole graph) * R, one launch per destination group, groups concurrently.
cudaError_t launch_fused(const sobek_plan* p, const Direction& dir, const EdgeView& ev, const float* src,
                         const float* vsrc, const float* Y, const float* vY, const float* phi, const float* vphi,
                         int dual, const void* fkh, const void* fkl, float* dst, int accumulate, int* status,
                         cudaStream_t s0) {
    const int KP = p->K <= 8 ? 8 : 16;
    const int US = 256 / KP, RW = 32 / US;
    Fork fork(p, s0);
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        FusedArgs a{};
        a.paths = dir.d_paths; a.stages = dir.d_fstages;
        a.tab_ptr = p->d_tab_ptr; a.tab_idx = p->d_tab_idx; a.tab_coef = p->d_tab_coef;
        a.G = G; a.fs_begin = dir.fs_begin[gi]; a.fs_count = dir.fs_count[gi];
        a.ev = ev; a.N = ev.N;
        a.src = src; a.vsrc = vsrc; a.Y = Y; a.vY = vY; a.phi = phi; a.vphi = vphi;
        a.dst = dst; a.C_src = dir.C_src; a.C_dst = dir.C_dst; a.accumulate = accumulate;
        a.K = p->K; a.dsh = p->dim_sh;
        a.NT = 128 / G.d_dst;
        a.BN = (G.c_dst + 15) / 16 * 16;
        int cols = 32;
        while (cols < a.BN) cols <<= 1;
        a.tmem_cols = cols;
        a.status = status;
        // M-stage pitch: max over the group's paths of d_src * OC
        const int OC = G.d_dst <= 5 ? G.d_dst : (G.d_dst == 7 ? 4 : 5);
        int ms = 4;
        for (int k = G.path_begin; k < G.path_end; ++k) ms = std::max(ms, (dir.paths[k].d_src * OC + 3) & ~3);
        if ((ms & 31) == 0) ms += 4;
        a.MS = ms;
        const size_t b_slab = (size_t)a.BN * 128;
        // shared memory: A tile (hi, lo) + B ring + barriers + producer stages; shrink the ring, then the
        // edge batch, until it fits
        size_t sh = 0;
        bool fits = false;
        for (int slots = (2 * b_slab * 4 <= 64 * 1024) ? 4 : 2; slots >= 2 && !fits; slots -= 2) {
            for (int eb = std::min(16, US); eb >= 2 && !fits; eb >>= 1) {
                int sf = eb * ms + eb * KP + eb * (a.dsh + 1) + 2 * eb;
                if (dual) sf += eb * ms + eb * KP + eb * (a.dsh + 1);
                sf = (sf + 3) & ~3;
                sh = 1024 + 2 * (size_t)A_BYTES_HOST + (size_t)slots * 2 * b_slab + 8 * (2 + 8 + 2 * slots) + 64 +
                     (size_t)8 * RW * sf * 4;
                if (sh <= 227 * 1024) { fits = true; a.nb_slots = slots; a.EB = eb; a.sub_floats = sf; }
            }
        }
        if (!fits) return cudaErrorInvalidValue;
        CUtensorMap th, tl;
        const int64_t ld = (int64_t)dir.fs_count[gi] * 256;
        const uint16_t* bh = (const uint16_t*)fkh + dir.fk_off[gi];
        const uint16_t* bl = (const uint16_t*)fkl + dir.fk_off[gi];
        if (!ptx::make_map(&th, bh, ld, G.c_dst, ld, 64, a.BN) || !ptx::make_map(&tl, bl, ld, G.c_dst, ld, 64, a.BN))
            return cudaErrorInvalidValue;
        const int grid = (int)((ev.N + a.NT - 1) / a.NT);
        cudaStream_t s = fork.pick();
        KernelTimer kt(K_FUSED, s);
        cudaError_t e;
        if (KP == 8) e = dual ? fused_launch_k8_dual(G.d_dst, th, tl, &a, grid, sh, s) : fused_launch_k8(G.d_dst, th, tl, &a, grid, sh, s);
        else e = dual ? fused_launch_k16_dual(G.d_dst, th, tl, &a, grid, sh, s) : fused_launch_k16(G.d_dst, th, tl, &a, grid, sh, s);
        count_launch();
        if (e != cudaSuccess) return e;
    }
    return fork.join();
}

}  // namespace sobek
