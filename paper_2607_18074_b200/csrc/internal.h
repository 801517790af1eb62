// Internal declarations shared by the translation units of libsobek (not installed).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <vector>

#include "sobek.h"

namespace sobek {

// ---------------------------------------------------------------------------------------
// Device-side description of one traversal direction.
//
// FORWARD direction:    destination groups = output irrep blocks, sources = input blocks of x.
// TRANSPOSED direction: destination groups = input irrep blocks (for gx), sources = output
//                       blocks of gy.  It is the same operator on the reversed graph with
//                       c'[m_out,m_sh,m_in] = c[m_in,m_sh,m_out] and R'[q,pi,w,u] = R[q,pi,u,w].
//
// For one edge and one path the angular contraction (Eq. angular_path_contraction) is split
// as  C[u,o] = sum_s xs[u,s] * M[s,o],  M[s,o] = sum_b coef * Y[b]: M depends on the edge and
// the path only, not on the multiplicity index, and is produced from the sparse table below.
// ---------------------------------------------------------------------------------------
struct DPath {
    int32_t src_off;   // offset of the source block inside a source feature row
    int32_t c_src;     // source multiplicity
    int32_t d_src;     // 2 l_src + 1
    int32_t sh_off;    // offset of the SH block inside a Y row
    int32_t d_sh;      // 2 l_sh + 1
    int32_t d_dst;     // 2 l_dst + 1
    int32_t c_dst;     // destination multiplicity
    int32_t koff;      // offset in the group's contraction axis; k = koff + q*c_src + u
    int32_t m_off;     // offset of M[s][o] inside the group's per-edge M area
    int32_t tabM;      // index into tab_ptr: entry (s*d_dst+o) -> terms (b, coef)
    int32_t tabY;      // index into tab_ptr: b -> terms (s*d_dst+o, coef)   (adjoint wrt Y)
    int32_t pad;
    int64_t rp_off;    // offset (floats) of the owning group's slab in the packed R
    int64_t w_off;     // first column of the path in R[K, N_w]
    int32_t c_in, c_out;  // multiplicities in the ORIGINAL orientation (column = u*c_out + w)
};

struct DGroup {
    int32_t dst_off;   // offset of the block inside a destination feature row
    int32_t c_dst;     // destination multiplicity (GEMM columns)
    int32_t d_dst;     // 2l+1 (rows per node)
    int32_t D;         // contraction width = K * sum c_src over the group's paths
    int32_t path_begin, path_end;
    int32_t m_entries; // sum over paths of d_src*d_dst
    int32_t wt_begin, wt_end;   // range in the warp-task list
    int32_t pad;
    int64_t z_off;     // offset (floats per node) of this group's state rows: sum_{g'<g} d*D
    int64_t rp_off;    // offset (floats) of this group's slab in the packed R: sum_{g'<g} D*c_dst
};

struct WTask {         // one warp's share of a group: 32 consecutive multiplicities of one path
    int32_t path;
    int32_t u0;
};

struct SComp {         // one output component handled by an edge-stream task
    int32_t tab0;      // tab_ptr index of the (s = 0, o) entry of the path's M table
    int32_t tstride;   // distance between consecutive s in that table (= d_dst of the path)
    int32_t sh_off;    // offset of the path's SH block inside a Y row
    int32_t group;     // destination group
    int32_t o;         // component inside the destination irrep
    int32_t koff;      // offset of the path in the group's contraction axis
    int32_t d_dst;     // 2l+1 of the destination group
    int32_t pad;
};

struct STask {         // one warp's task of the edge stream (source-major)
    int32_t src_off;   // offset of the source block inside a source feature row
    int32_t c_src;     // source multiplicity
    int32_t d_src;     // 2l+1 of the source
    int32_t u0;        // first of the 32 multiplicities of the task
    int32_t ncomp;     // output components of the task
    int32_t comp_begin;
    int32_t cls;       // kernel class: padded d_src (0: <=3, 1: <=5, 2: <=9)
    int32_t pad;
};

// --- tensor-core edge stream (stream_tc.cu) ------------------------------------------------
// Per receiver and source irrep block the fold over its edges is the dense contraction
//     Z[(comp,q), u] = sum_{(e,s)} ( phi_e[q] * M_e[s,comp] ) * x_{src(e)}[s,u]
// A "unit" is one accumulator tile of it: up to 128 rows (comp,q) of one source block.  A "set" is
// the group of units one CTA pass holds at once (bounded by shared memory and TMEM columns).
struct TEnt {          // one (unit, component, s) entry of a set: a row block of one A slab
    int32_t tab;       // tab_ptr index of the entry's sparse terms (b, coef)
    int32_t sh_off;    // offset of the path's SH block inside a Y row
    int32_t a_off;     // byte offset of row (component*KP) of slab s inside one A copy
    int32_t pad;
};
struct TUnit {
    int32_t blk;           // index into the block list
    int32_t comp_begin;    // first component (index into the TC component list)
    int32_t ncomp;
    int32_t a_off;         // byte offset of the unit's slab 0 inside one A copy
    int32_t slab_stride;   // bytes between consecutive s slabs of the unit
    int32_t tmem_col;      // first accumulator column
    int32_t pad[2];
};
struct TBlk {
    int32_t src_off, c_src, d_src;
    int32_t ncols;         // accumulator columns = c_src rounded up to 16
    int32_t b_off;         // byte offset of the block's slab 0 inside one B copy
    int32_t slab_bytes;    // bytes between consecutive s slabs of the gathered rows
    int32_t atom_stride;   // bytes between the 64-multiplicity column blocks of a slab
    int32_t pad;
};
struct TSet {
    int32_t unit_begin, nunit, blk_begin, nblk, ent_begin, nent;
    int32_t b_items;       // float4 pieces of sender rows gathered per 16-edge batch
    int32_t pad;
    // stream: the set's slab list (TcSets::slabs, two words per slab), slabs per batch, first slab of each MMA thread
    // (one byte each, 255: none) and the slots that a batch uses an odd number of times
    int32_t sched_begin, nslab, mfirst, oddmask;
};
struct EntS {          // a (unit, component, s) entry of a set, as the kernels keep it in shared memory
    int32_t a_off, nz_begin, nz_count, pad;   // nz_begin is relative to the set's first term
};
struct NzS {           // one sparse CG term of an entry: Y index and coefficient
    int32_t b;
    float coef;
};
struct CompS {         // an output component with the layout of its destination group resolved
    int64_t zoff;      // bf16 state offset per node of the group
    int32_t ld, d_dst, o, koff;
    int32_t pad[2];
};
struct TcSets {
    bool ok = false;       // the tensor-core stream supports this direction
    std::vector<TSet> sets;
    std::vector<TUnit> units;
    std::vector<TBlk> blks;
    std::vector<TEnt> ents;
    std::vector<SComp> comps;
    TSet* d_sets = nullptr;
    TUnit* d_units = nullptr;
    TBlk* d_blks = nullptr;
    TEnt* d_ents = nullptr;
    SComp* d_comps = nullptr;
    std::vector<EntS> ents_s;                // per set (TSet::ent_begin); TSet::b_items / TSet::pad = first term / terms
    std::vector<NzS> nz;
    std::vector<CompS> comps_s;              // parallel to comps
    std::vector<uint32_t> slabs;             // stream: per set, two words per slab in build order (see stream_tc.cu)
    uint32_t* d_slabs = nullptr;
    EntS* d_ents_s = nullptr;
    NzS* d_nz = nullptr;
    CompS* d_comps_s = nullptr;
    int32_t max_nz = 0;
    std::vector<int32_t> inv_ptr, inv_base;  // edge pass: per set, dsh+1 relative offsets / first term of the set
    std::vector<NzS> inv;                    //   b -> terms (entry inside the set, coef)
    int32_t* d_inv_ptr = nullptr;
    NzS* d_inv = nullptr;
    int32_t max_units = 0;                   // stream: slabs of a batch that one builder group builds, at most
    struct ESetPar { int32_t tb, lg, x_cap, z_cap, smem, ctas, tmem_cols, acc_cols, nnz, ninv, ncomp; };
    std::vector<ESetPar> epar;               // edge pass: launch parameters of every set (one launch per set)
    int32_t a_cap = 0, b_cap = 0;     // bytes of one A / B copy (max over sets; the stream keeps A in tensor memory)
    int32_t max_ent = 0, tmem_cols = 32;
    int32_t acc_cols = 0;             // accumulator columns of one buffer (two buffers are allocated)
    int32_t ring_stages = 2;          // stream: stages of the shared-memory ring (as many as fit)
    int32_t nbuf = 2;                 // stream: accumulator buffers in tensor memory (2, or 1 for wider sets)
    int32_t smem_bytes = 0, ctas_per_sm = 1;
};

struct FStage {        // one 256-column stage of the fused kernel's contraction axis
    int32_t path;
    int32_t u0;        // first multiplicity of the block (256/KP wide)
    int32_t q0;        // first radial component (0 unless K > 16)
    int32_t group;
};

struct Direction {
    // host copies
    std::vector<DPath> paths;
    std::vector<DGroup> groups;
    std::vector<WTask> wtasks;
    int64_t state_floats = 0;   // per node: sum_g d*D
    int32_t max_m_entries = 0;
    int32_t C_src = 0, C_dst = 0;
    // bf16 operand layouts (element offsets / leading dimensions per group; groups without paths get 0)
    //   KN: [k][c_dst], ld = round8(c_dst)   NK: [c_dst][k], ld = round8(D)
    std::vector<int64_t> kn_off, nk_off;
    std::vector<int32_t> kn_ld, nk_ld, path_group;
    int64_t kn_elems = 0, nk_elems = 0;
    std::vector<int64_t> zb_off;      // per node, elements: sum_{g'<g} d * round8(D)     (bf16 state rows)
    std::vector<int64_t> gb_off;      // per node, elements: sum_{g'<g} d * round8(c_dst) (bf16 adjoint rows)
    int64_t zb_elems = 0, gb_elems = 0;
    std::vector<STask> stasks;        // sorted by kernel class
    std::vector<SComp> scomps;
    struct SClass { int cls, begin, count; };
    std::vector<SClass> sclasses;
    STask* d_stasks = nullptr;
    SComp* d_scomps = nullptr;
    TcSets tc[2];                     // tensor-core stream: [0] plain, [1] dual
    TcSets etc[2];                    // tensor-core edge pass: [0] plain, [1] dual
    // receiver-owned edge pass: source-major tasks over all multiplicities
    std::vector<STask> etasks;
    std::vector<SComp> ecomps;
    std::vector<SClass> eclasses;
    STask* d_etasks = nullptr;
    SComp* d_ecomps = nullptr;
    int64_t* d_zb_off = nullptr;
    // fused kernels: stage list, per-group ranges and the stage-ordered bf16 copy of R
    std::vector<FStage> fstages;
    std::vector<int32_t> fs_begin, fs_count;
    std::vector<int64_t> fk_off;
    int64_t fk_elems = 0;
    FStage* d_fstages = nullptr;
    int32_t *d_fs_begin = nullptr, *d_fs_count = nullptr;
    int64_t* d_fk_off = nullptr;
    // device copies
    DPath* d_paths = nullptr;
    DGroup* d_groups = nullptr;
    WTask* d_wtasks = nullptr;
    int64_t *d_kn_off = nullptr, *d_nk_off = nullptr;
    int32_t *d_kn_ld = nullptr, *d_nk_ld = nullptr, *d_path_group = nullptr;
};

struct HPath {
    sobek_path_info info;
    std::vector<double> cg;   // dense [d_in][d_sh][d_out]
};

}  // namespace sobek

// Direct forward of the channelwise mode (uvu_direct.cu): tables in the kernel's static path order
struct UvuDirectTables {
    std::vector<int32_t> woff;      // per path: first weight column
    std::vector<int2> ent;          // per stored coupling-matrix entry: {offset in the padded M_e | terms << 16, first term}
    std::vector<int2> nz;           // sparse terms: {index into a Y row, coefficient bits}
    int32_t* d_woff = nullptr;
    int2* d_ent = nullptr;
    int2* d_nz = nullptr;
};
struct UvuDirect {
    bool ok = false;
    int L = 0, C = 0, H = 1;        // H: channel slices, one CTA each (C / H channels x thread shares <= 256 threads)
    UvuDirectTables dir[2];         // [0] y from x on the receiver view, [1] gx from gy on the sender view
};

struct sobek_plan {
    std::vector<sobek_irrep> in, out;
    int l_max = 0, K = 0;
    int C_x = 0, C_y = 0, dim_sh = 0;
    int64_t N_w = 0;
    std::vector<sobek::HPath> paths;
    sobek::Direction fwd, tr;
    // sparse tables (shared by both directions)
    std::vector<int32_t> tab_ptr;
    std::vector<int32_t> tab_idx;
    std::vector<float> tab_coef;
    int32_t* d_tab_ptr = nullptr;
    int32_t* d_tab_idx = nullptr;
    float* d_tab_coef = nullptr;
    int device = -1;
    bool use_tc_stream = true;   // edge stream on the tensor cores where the profile allows it
    bool use_tc_edge = true;     // edge pass on the tensor cores where the profile allows it
    size_t state_budget = size_t(2048) << 20;   // bytes of receiver / sender state held at once (the scratch budget)
    int gemm_passes = 3;      // 3: split-bf16 node GEMMs (fp32-faithful); 1: plain bf16 GEMMs (SOBEK_FLAG_FAST_GEMM)
    bool mul_ir = false;      // node features cross the boundary in mul_ir order and are re-laid through the workspace
    int4* d_in_blocks = nullptr;    // {offset, multiplicity, 2l+1, 0} of the irrep blocks of x / of y (device), for the re-layout
    int4* d_out_blocks = nullptr;
    bool uvu = false;         // channelwise mode (Eq. uvu_connection): tied multiplicities, C_in weights per path
    UvuDirect ud;             // its direct kernel (y and gx), where the profile allows it
    bool uvu_state = false;   // SOBEK_FLAG_UVU_STATE: through the receiver state even so
    bool use_fused = false;   // schedule choice: fused stream+contraction kernels vs. stream -> state -> GEMM
    // side streams used to run independent kernels of one call concurrently (joined back into the
    // caller's stream before the call returns control of ordering)
    static constexpr int kSide = 4;
    cudaStream_t side[kSide] = {};
    cudaEvent_t ev_fork = nullptr;
    cudaEvent_t ev_join[kSide] = {};
    int n_side = 0;
};

namespace sobek {

// bytes reserved at the start of every workspace for the device status word
constexpr size_t kHeaderBytes = 256;
// budget for the bounded node-state buffer (floats of Z / V held at once)
constexpr int64_t kMinChunkNodes = 512;

int64_t chunk_nodes(const sobek_plan* p, int64_t N, int order);

void count_launch(int n = 1);

// Fork/join of the caller's stream into the plan's side streams: kernels launched on pick() run
// concurrently with each other and are all ordered after what was queued on `main` before the
// fork and before what is queued on `main` after join().
class Fork {
public:
    Fork(const sobek_plan* p, cudaStream_t main);
    cudaStream_t pick();
    cudaError_t join();
private:
    const sobek_plan* p_;
    cudaStream_t main_;
    int used_ = 0;
    bool on_ = false;
};

enum KernelClass { K_PACK = 0, K_STATE, K_GEMM, K_EDGE, K_FILL, K_FUSED, K_NCLASS };
// Brackets one launch with CUDA events when timing is enabled (sobek_timing_enable).
class KernelTimer {
public:
    KernelTimer(int cls, cudaStream_t s);
    ~KernelTimer();
private:
    int cls_;
    cudaStream_t s_;
    bool on_;
    cudaEvent_t a_{}, b_{};
};

// --- kernels.cu ---------------------------------------------------------------------
struct EdgeView {          // how a traversal walks the graph
    const int64_t* ptr;    // [N+1] segment pointers of the owning node
    const int32_t* perm;   // NULL: position == edge id; else edge id = perm[position]
    const int32_t* col;    // sender of each edge (edge-id indexed)
    const int64_t* row_ptr;// receiver CSR (to recover the receiver of an edge id)
    int64_t N, E;
    int transposed;        // 0: source node = col[e];  1: source node = receiver(e)
    const int32_t* recv;   // transposed only, optional: receiver of the edge at each position (else searched)
};

cudaError_t launch_unpack_R(const sobek_plan* p, const Direction& dir, const float* Rp, float* R,
                            cudaStream_t s);
void build_edge_tasks(const sobek_plan* p, Direction& dir);
// receiver-owned edge pass: gphi_e = <Zbar, C_e>, gY_e = CG^T_Y(x, phi_e Zbar); with `dual` the
// second-order terms that share Zbar: <Zbar, C(vx,Y)+C(x,vY)> and CG^T_Y(vx, phi Zbar) + CG^T_Y(x, vphi Zbar)
cudaError_t launch_edge_pass(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                             int64_t n_nodes, const float* src, const float* vsrc, const float* Y, const float* vY,
                             const float* phi, const float* vphi, int dual, const float* Zbar, float* gphi,
                             float* gY, int phi_mode, int Y_mode /* 0 skip, 1 overwrite, 2 accumulate */,
                             int* status, cudaStream_t s);
cudaError_t launch_fill_zero(float* p, int64_t n, cudaStream_t s);
// [N][C] node features between the two block orders: to_ir_mul = 1: dst[m*C_b + u] = src[u*d + m] inside every block
cudaError_t launch_relayout(const float* src, float* dst, int64_t N, int C, const int4* blocks, int nblk, int to_ir_mul,
                            cudaStream_t s);

// --- edge_stream.cu ---------------------------------------------------------------
void build_stream_tasks(const sobek_plan* p, Direction& dir);
// bf16 (hi, lo) copies of the source features of a traversal, [N][C_src] each (made once per call);
// all NULL when the caller has none (the FP32-pipe stream is used then)
struct SplitSrc {
    const void* h = nullptr;
    const void* l = nullptr;
    const void* vh = nullptr;   // the same for the source direction of the dual stream (NULL without it)
    const void* vl = nullptr;
    // geometry mode of the tensor-core edge kernels: edge vectors [E][3] from which Y and phi are recomputed (the Y and
    // phi arguments are NULL then), and where the edge pass puts the adjoint of the edge vectors instead of gY, gphi
    const float* rvec = nullptr;
    float geo_rc = 0.f;
    int geo_basis = 0, geo_p = 6;
    float* g_rvec = nullptr;
    const float* vrvec = nullptr;     // double backward: direction on the edge vectors (dual stream passes only)
    // load balance of the tensor-core edge kernels: [N] entries {local node, segment begin, segment end, 0}, the nodes of
    // every chunk in the order its persistent CTAs take them (launch_chunk_order); NULL: index order
    const int4* oseg = nullptr;
};
cudaError_t launch_stream(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                          int64_t n_nodes, const float* src, const float* vsrc, const SplitSrc& ss, const float* Y,
                          const float* vY, const float* phi, const float* vphi, int dual, void* zh, void* zl,
                          int* status, cudaStream_t s);
// --- edge_pass_tc.cu ------------------------------------------------------------------
void build_tc_edge_sets(const sobek_plan* p, Direction& dir);
cudaError_t launch_edge_pass_tc(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                                int64_t n_nodes, const SplitSrc& ss, const float* Y, const float* vY, const float* phi,
                                const float* vphi, int dual, const void* zqh, const void* zql, float* gphi, float* gY,
                                int phi_mode, int Y_mode, int* status, cudaStream_t s);
// --- stream_tc.cu ---------------------------------------------------------------------
void build_tc_sets(const sobek_plan* p, Direction& dir);
cudaError_t launch_stream_tc(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                             int64_t n_nodes, const SplitSrc& ss, const float* Y, const float* vY, const float* phi,
                             const float* vphi, int dual, void* zh, void* zl, int* status, cudaStream_t s);

cudaError_t stream_launch_k8(const void* args, int cls, int t_begin, int t_count, cudaStream_t s);
cudaError_t stream_launch_k16(const void* args, int cls, int t_begin, int t_count, cudaStream_t s);
cudaError_t stream_launch_k8_dual(const void* args, int cls, int t_begin, int t_count, cudaStream_t s);
cudaError_t stream_launch_k16_dual(const void* args, int cls, int t_begin, int t_count, cudaStream_t s);

// --- fused.cu -------------------------------------------------------------------------
struct FusedArgs {   // arguments of the fused kernels (fused_impl.cuh)
    const DPath* paths;
    const FStage* stages;
    const int32_t* tab_ptr;
    const int32_t* tab_idx;
    const float* tab_coef;
    DGroup G;
    int32_t fs_begin, fs_count;
    EdgeView ev;
    int64_t N;
    const float* src;
    const float* vsrc;
    const float* Y;
    const float* vY;
    const float* phi;
    const float* vphi;
    float* dst;
    int32_t C_src, C_dst, accumulate;
    int32_t K, dsh;
    int32_t NT;          // nodes per tile = 128 / D
    int32_t BN;          // padded destination multiplicity (multiple of 16)
    int32_t tmem_cols;
    int32_t nb_slots;    // B ring slots
    int32_t EB;          // edges staged per batch (<= 16, <= multiplicities per stage)
    int32_t MS;          // row pitch of the M stage
    int32_t sub_floats;  // shared floats of one node's staging area (one per node handled by a warp)
    int* status;
};

constexpr size_t A_BYTES_HOST = 4 * 128 * 128;   // one of (hi, lo) of the 128 x 256 bf16 A tile
void build_fused_stages(const sobek_plan* p, Direction& dir);
bool fused_supported(const sobek_plan* p, const Direction& dir);
cudaError_t launch_pack_R_fused(const sobek_plan* p, const Direction& dir, int transposed, const float* R, void* hi,
                                void* lo, cudaStream_t s);
cudaError_t launch_fused(const sobek_plan* p, const Direction& dir, const EdgeView& ev, const float* src,
                         const float* vsrc, const float* Y, const float* vY, const float* phi, const float* vphi,
                         int dual, const void* fkh, const void* fkl, float* dst, int accumulate, int* status,
                         cudaStream_t s0);
#define SOBEK_FUSED_DECL(name)                                                                              \
    cudaError_t name(int D, const CUtensorMap& th, const CUtensorMap& tl, const void* args, int grid, size_t sh, \
                     cudaStream_t s)
SOBEK_FUSED_DECL(fused_launch_k8);
SOBEK_FUSED_DECL(fused_launch_k8_dual);
SOBEK_FUSED_DECL(fused_launch_k16);
SOBEK_FUSED_DECL(fused_launch_k16_dual);

// --- gemm_tc.cu ---------------------------------------------------------------------
int64_t round8(int64_t v);
// the packings of R (or of its direction vR) into GEMM operand layouts that one call needs, queued and run as one launch
struct PackJob {
    const DPath* paths; const int64_t* grp_off; const int32_t* grp_ld; const int32_t* path_group;
    int n_paths, transposed, n_major;
    const float* R; void* hi; void* lo;
};
constexpr int kMaxPackJobs = 6;
struct PackQueue {
    const sobek_plan* p;
    PackJob j[kMaxPackJobs];
    int n = 0;
    bool overflow = false;
    explicit PackQueue(const sobek_plan* plan) : p(plan) {}
    // n_major = 1: [c_dst][k] rows (B operand of y = Z Rp); 0: [k][c_dst] rows (B operand of Zbar = gy Rp^T); no-op in
    // the channelwise mode, which has no operand copies
    void add(const Direction& dir, int transposed, int n_major, const float* R, void* hi, void* lo);
    cudaError_t flush(cudaStream_t s);
};
// several fp32 -> (bf16 hi, lo) conversions with mapped source rows in one launch (see launch_split)
struct SplitJob { const float* src; int64_t s_outer, s_inner; int s_d; int64_t rows; int cols; int64_t ld; void* hi; void* lo; };
constexpr int kMaxSplitJobs = 8;
cudaError_t launch_split_jobs(const SplitJob* jobs, int n, cudaStream_t s);
cudaError_t launch_split(const float* src, int64_t s_outer, int64_t s_inner, int s_d, int64_t rows, int cols,
                         int64_t ld, void* hi, void* lo, cudaStream_t s);
cudaError_t launch_pack_R_bf16(const sobek_plan* p, const Direction& dir, int transposed, int n_major,
                               const float* R, void* hi, void* lo, cudaStream_t s);
// a queue of tensor-core products that one launch runs (gemm_tc.cu); plain storage so that only gemm_tc.cu needs the
// tensor-map type
struct GemmBatch {
    alignas(64) unsigned char storage[4096];
    size_t sh = 0;      // dynamic shared memory the queued products need (the largest)
    size_t sh_of[8] = {};   // and each of them
    int n = 0;
};
cudaError_t gemm_tc_add(GemmBatch& gb, const void* Ahi, const void* Alo, int64_t lda, const void* Bhi, const void* Blo,
                        int64_t ldb, float* C, int64_t c_outer, int64_t c_inner, int c_d, int64_t M, int64_t N,
                        int64_t Kd, int accumulate, int mn_major, int* status, cudaStream_t s, int splits,
                        int64_t split_stride, void* Chi, void* Clo, int passes);
// p: the plan whose side streams carry the products when they are launched one by one (NULL: all on s)
cudaError_t gemm_tc_flush(GemmBatch& gb, cudaStream_t s, const sobek_plan* p);
cudaError_t launch_gemm_tc(const void* Ahi, const void* Alo, int64_t lda, const void* Bhi, const void* Blo,
                           int64_t ldb, float* C, int64_t c_outer, int64_t c_inner, int c_d, int64_t M, int64_t N,
                           int64_t Kd, int accumulate, int mn_major, int* status, cudaStream_t s, int splits = 1,
                           int64_t split_stride = 0, void* Chi = nullptr, void* Clo = nullptr, int passes = 3);
cudaError_t launch_reduce_parts(float* dst, const float* part, int64_t n, int64_t stride, int splits, cudaStream_t s);
// the same for several column ranges of one [splits][stride] buffer in one launch: dst[off + i] += sum_z part[z][off + i]
struct ReduceRange { int64_t off, n; int splits; };
constexpr int kMaxReduceRanges = 8;
cudaError_t launch_reduce_ranges(float* dst, const float* part, int64_t stride, const ReduceRange* r, int nr, cudaStream_t s);
cudaError_t launch_wait_selftest(int* status, uint64_t limit_ns, cudaStream_t s);
constexpr int kMaxSplits = 8;                                  // split-K pieces of the weight-adjoint GEMM
constexpr size_t kPartBudgetBytes = size_t(64) << 20;          // bound on its partial-result buffer

// --- geometry_second.cu: second-order geometry by hyper-dual evaluation of the bases --------------------
bool geo_second_supported(int l_max, int K);
cudaError_t launch_geo_edge_inputs(const float* rvec, const float* vrvec, int64_t E, int l_max, int K, float r_c, int basis, int p,
                                   float* Y, float* phi, float* vY, float* vphi, cudaStream_t s);
cudaError_t launch_geo_second_adjoint(const float* rvec, const float* vrvec, int64_t E, int l_max, int K, float r_c, int basis,
                                      int p, const float* gY, const float* gphi, const float* hY, const float* hphi,
                                      float* h_rvec, cudaStream_t s);
// For every chunk of `chunk` nodes of the view: its nodes sorted by segment length, longest first, dealt in rounds of
// `period` that alternate direction, so that CTAs taking the entries round-robin get equal shares of the edges.
cudaError_t launch_chunk_order(const EdgeView& ev, int64_t chunk, int period, int4* oseg, int* status, cudaStream_t s);
// --- uvu_direct.cu ------------------------------------------------------------------------
void build_uvu_direct(sobek_plan* p, const sobek_irrep* in, int n_in, const sobek_irrep* out, int n_out);
// transposed = 0: y[N, C_y] from src = x on the receiver view; 1: gx[N, C_x] from src = gy on the sender view
cudaError_t launch_uvu_direct(const sobek_plan* p, const EdgeView& ev, int transposed, const float* src, const float* Y,
                              const float* phi, const float* R, float* dst, int* status, cudaStream_t s);
// part[0 .. *n_parts)[K * N_w]: per-CTA sums of the weight adjoint gR over the receivers (receiver view only)
cudaError_t launch_uvu_direct_wgrad(const sobek_plan* p, const EdgeView& ev, const float* x, const float* Y, const float* phi,
                                    const float* gy, float* part, int max_parts, int* n_parts, int* status, cudaStream_t s);
// --- node_uvu.cu: the node-side steps of the channelwise mode (no GEMM) ---------------
cudaError_t launch_uvu_mix(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const void* zh,
                           const void* zl, const float* R, float* dst, int accumulate, cudaStream_t s0);
cudaError_t launch_uvu_zbar(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const float* gy,
                            const float* R, float* Zbar, void* zqh, void* zql, cudaStream_t s0);
cudaError_t launch_uvu_wgrad(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const void* zh,
                             const void* zl, const float* gy, float* gR_acc, float* part, int splits,
                             cudaStream_t s0);
constexpr int kMaxSplitsUvu = 512;                             // node slices of the channelwise weight adjoint

// --- graph.cu -----------------------------------------------------------------------
size_t graph_prepare_bytes(int64_t N, int64_t E);
int graph_receivers(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* src_perm, int32_t* src_recv,
                    cudaStream_t s);
int edge_vectors(const sobek_graph* g, const float* pos, float* rvec, cudaStream_t s);
int position_gradient(const sobek_graph* g, const float* g_rvec, float* gpos, cudaStream_t s);
int graph_prepare(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* col, int64_t* src_ptr,
                  int32_t* src_perm, void* ws, size_t ws_bytes, cudaStream_t s);

}  // namespace sobek
