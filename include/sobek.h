/*
 * sobek.h -- C ABI of the streaming edge-conditioned tensor-product convolution
 * (fully connected `uvw` multiplicity mixing) for NVIDIA B200 (sm_100a).
 *
 * The operator (Eq. standard_tpconv_background with W = phi A, Eq. edge_weight_shape;
 * the radial projection A is called R here):
 *
 *     y_i = sum_{j in N(i)} sum_pi sum_{u,w} ( sum_q phi_ij[q] R[q,pi,u,w] ) *
 *                 sum_{m_in,m_sh} c^pi[m_in,m_sh,m_out] x_j[pi,u,m_in] Y_ij[pi,m_sh]
 *
 * evaluated in the receiver-factorised streaming order (Eqs. angular_path_contraction,
 * receiver_state, receiver_mixing): each edge's CG coupling is scaled by phi_ij and
 * folded into a bounded per-receiver state Z_i, and Z_i is contracted with R.  No
 * array with |E| x N_w or |E| x C_out elements is ever formed, in any order of
 * differentiation.
 *
 * Conventions
 *   - All array arguments of the sobek_conv_* / sobek_graph_prepare calls are DEVICE
 *     pointers owned by the caller and must stay valid until the work queued on
 *     `stream` (a cudaStream_t passed as void*; NULL = default stream) has finished.
 *     Every floating-point array must start on a 16-byte boundary (the kernels copy 16-byte pieces of
 *     phi / vphi rows and of feature rows); a pointer that does not is refused with INVALID_ARG.
 *     Plan handles and descriptor arrays are HOST memory.
 *   - fp32 data, row-major.  Node features x[N,C_x], y/gy/ggy[N,C_y] use the `ir_mul`
 *     layout (Section "Generated deterministic runtime and execution contracts"):
 *     irrep blocks in descriptor order; inside a block the index is m*mult + u with
 *     m = 0..2l (standing for -l..l).  Y, gY, vY, hY are [E,(l_max+1)^2], l-major.
 *     phi, gphi, vphi, hphi are [E,K].  R, gR, vR, hR are [K,N_w] with column
 *     w_off(pi) + u*C_out(pi) + w; paths pi are numbered in nested order (input
 *     irrep, SH order, output irrep).
 *   - Real spherical-harmonic basis with sine-type components at m < 0 (l = 1 is
 *     (y,z,x)); c^pi = sqrt(2 l_out+1) x (unit-norm real 3j tensor whose first nonzero
 *     entry in lexicographic (m_in,m_sh,m_out) order is positive).
 *   - Graph: receiver-sorted CSR.  Edge e in [row_ptr[i], row_ptr[i+1]) runs from
 *     sender col[e] to receiver i; the order inside a row is the caller's and is kept.
 *     Empty rows, self loops and duplicate edges are legal.
 *   - Every entry point returns 0 on success or a negative sobek_status.  Nothing
 *     throws.  The sobek_conv_* calls never allocate device memory and never
 *     synchronise: they only enqueue work on `stream` and on side streams owned by the
 *     plan that are forked from and joined back into `stream` with events (so the call
 *     is ordered like a single kernel on `stream`).  Two calls using the same plan must
 *     not be issued concurrently from different host threads.  Results are bitwise
 *     reproducible from run to run (fixed reduction order, no floating-point atomics).
 *   - Outputs are overwritten, never accumulated into.  A NULL output pointer means
 *     "not wanted"; a NULL direction pointer in sobek_conv_dbwd means zero.
 */
#ifndef SOBEK_H_
#define SOBEK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SOBEK_OK = 0,
    SOBEK_ERR_INVALID_ARG = -1,    /* null pointer, negative size, bad descriptor            */
    SOBEK_ERR_UNSUPPORTED = -2,    /* l above the supported maximum, no valid path, ...     */
    SOBEK_ERR_WORKSPACE = -3,      /* workspace missing, misaligned or too small            */
    SOBEK_ERR_GRAPH = -4,          /* row_ptr not monotone / col out of range               */
    SOBEK_ERR_NEED_TRANSPOSE = -5, /* gx / hx wanted but src_ptr / src_perm are NULL        */
    SOBEK_ERR_CUDA = -6,           /* a CUDA runtime call or a launch failed                */
    SOBEK_ERR_DEVICE_TIMEOUT = -7  /* a bounded device-side wait gave up                    */
} sobek_status;

/* One irrep block of a feature vector: `mul` copies of order l with parity +1 (e) / -1 (o). */
typedef struct {
    int32_t mul;
    int32_t l;
    int32_t parity;
} sobek_irrep;

typedef struct sobek_plan sobek_plan; /* opaque; host-owned; immutable after creation */

enum { SOBEK_MAX_L = 4 };

/* plan flags */
#define SOBEK_FLAG_UVU 1u      /* channelwise multiplicity mode, Eq. uvu_connection */
#define SOBEK_FLAG_MUL_IR 2u   /* node features cross the boundary in mul_ir order (see sobek_plan_create) */
#define SOBEK_FLAG_FAST_GEMM 4u /* node-side GEMMs as plain bf16 products: lower precision, optional */
#define SOBEK_FLAG_FUSED_FP32 8u   /* schedule: FP32-pipe edge stream feeding the tensor core inside one kernel */
#define SOBEK_FLAG_FP32_STREAM 16u /* edge stream on the FP32 pipes even where the tensor-core kernel applies */
#define SOBEK_FLAG_FP32_EDGE 32u   /* edge pass on the FP32 pipes even where the tensor-core kernel applies */
#define SOBEK_FLAG_UVU_STATE 64u   /* channelwise mode: y and gx through the receiver state even where the direct kernel applies */
/* scratch budget in MiB (1 .. 2^20 - 1) in bits 12..31 of the flags word; 0 = the default */
#define SOBEK_FLAG_STATE_BUDGET_MIB(mb) (((uint32_t)(mb) & 0xFFFFFu) << 12)

/*
 * sobek_plan_create -- the static contract of one layer (Section "Generated
 * deterministic runtime and execution contracts"): enumerates the paths allowed by the
 * selection rules (Eq. cg_selection_rules) for spherical harmonics 1 x l, parity (-1)^l,
 * l = 0..l_max, computes the real Clebsch-Gordan tensors and uploads the sparse tables to
 * the current CUDA device (the only device allocation the library ever makes; it is
 * released by sobek_plan_destroy).  `in`/`out` are host arrays.  K >= 1 is the width of
 * the radial embedding.  `flags` is 0 for fully connected multiplicity mixing (Eq. uvw_connection:
 * C_in*C_out weights per path, column w_off + u*C_out + w of R) or SOBEK_FLAG_UVU for the channelwise
 * mode (Eq. uvu_connection: output multiplicity tied to the input one, C_in weights per path, column
 * w_off + u; N_w = sum of C_in over the paths; a path between blocks of different multiplicity makes the
 * call fail with UNSUPPORTED).  Every other argument, layout and entry point is the same in both modes.
 * SOBEK_FLAG_MUL_IR (may be combined with the above) selects the mul_ir order for every node feature array
 * at the boundary (x, y, gy, gx, vx, ggy, hx): inside an irrep block of multiplicity C the element (u, m) sits at
 * u*(2l+1) + m instead of m*C + u (Section "Generated deterministic runtime and execution contracts": the kernels
 * work in ir_mul, the other order is transposed at the boundary).  The calls then re-lay the arrays through the
 * workspace, which grows by 4 bytes per node feature and array; Y, phi and R are unaffected.
 * SOBEK_FLAG_FAST_GEMM replaces the three-pass split-bf16 product of the node-side GEMMs (fp32-faithful, the default
 * and what every stated tolerance refers to) by the single bf16 product a_hi*b_hi with fp32 accumulation: the optional
 * reduced-precision channel GEMM of the paper's runtime contract.  Relative errors of about 1e-2 of the largest output
 * are to be expected; the edge kernels keep their three-pass products; the flag has no effect in the uvu mode.
 * SOBEK_FLAG_FUSED_FP32 selects the fused schedule for y / gx / ggy / hx (FP32-pipe edge stream feeding the tensor
 * core inside one kernel, receiver state never written to memory); the default is the stream -> bounded state ->
 * GEMM schedule, which is the faster one at present.  In the default schedule the edge stream and the edge pass run
 * on the tensor cores where the profile allows it (multiplicities that are multiples of 8 / 16, at most 128,
 * K <= 16); SOBEK_FLAG_FP32_STREAM / SOBEK_FLAG_FP32_EDGE select the FP32-pipe kernels instead (same results
 * within the tolerances).
 * SOBEK_FLAG_STATE_BUDGET_MIB(mb) sets the scratch budget (section "Runtime scratch-budget policy"; the paper
 * measures with 128 MiB): the bytes of receiver (or sender) state held at once.  Nodes are processed in chunks that
 * fit the budget, but never fewer than 512 at a time; the results do not depend on the budget beyond the summation
 * order of gR / hR across chunks.  Without it the budget is 2048 MiB.
 * Errors: INVALID_ARG (null, mul < 1, parity not +-1, K < 1), UNSUPPORTED (l or l_max >
 * SOBEK_MAX_L, or no valid path), CUDA.
 */
int sobek_plan_create(const sobek_irrep* in, int n_in, const sobek_irrep* out, int n_out,
                      int l_max, int K, uint32_t flags, sobek_plan** plan);
void sobek_plan_destroy(sobek_plan* plan);

typedef struct {
    int32_t C_x;     /* flattened input width  (Eq. flattened_feature_dimension) */
    int32_t C_y;     /* flattened output width                                   */
    int32_t dim_sh;  /* (l_max+1)^2                                              */
    int32_t K;
    int32_t n_paths;
    int32_t l_max;
    int64_t N_w;     /* Eq. num_weights                                          */
    int64_t state_floats_fwd; /* K*F : floats of receiver state Z per node       */
    int64_t state_floats_bwd; /* K*F': floats of sender state V per node         */
} sobek_info;

typedef struct {
    int32_t i_in, l_sh, i_out;   /* input irrep index, SH order, output irrep index */
    int32_t l_in, l_out;
    int32_t c_in, c_out;         /* coupled multiplicities: n_pi = c_in*c_out       */
    int32_t in_off, sh_off, out_off; /* offsets inside an x row, a Y row, a y row   */
    int64_t w_off;               /* first column of this path in R                  */
} sobek_path_info;

int sobek_plan_info(const sobek_plan* plan, sobek_info* info);
int sobek_plan_path(const sobek_plan* plan, int path, sobek_path_info* info);
/* Dense c^pi[m_in][m_sh][m_out] (host, (2l_in+1)(2l_sh+1)(2l_out+1) doubles) as the library
 * computed it (Eq. angular_path_contraction); for inspection and tests. */
int sobek_plan_cg(const sobek_plan* plan, int path, double* dense);

/*
 * Graph in receiver-sorted CSR form plus its sender-sorted view ("cached stable CSR
 * views", Section "Generated deterministic runtime and execution contracts").
 */
typedef struct {
    int64_t N, E;
    const int64_t* row_ptr;  /* [N+1] row_ptr[0] = 0, row_ptr[N] = E, non-decreasing        */
    const int32_t* col;      /* [E]   sender of each edge                                   */
    const int64_t* src_ptr;  /* [N+1] sender-sorted view; may be NULL if gx/hx not wanted   */
    const int32_t* src_perm; /* [E]   edge ids grouped by sender, increasing inside a group */
    const int32_t* src_recv; /* [E]   optional: receiver of edge src_perm[p] at position p (see
                                      sobek_graph_receivers); NULL = looked up in row_ptr when needed */
} sobek_graph;

/*
 * sobek_graph_prepare -- validates (row_ptr, col) and builds the stable sender-sorted view
 * used by the source-owned traversal of the backward passes (Section "Receiver-factorized
 * backward").  Integer work; the result is unique, so it can be compared bit for bit.
 * `ws` needs sobek_graph_prepare_bytes(N, E) bytes, 256-byte aligned.  This call
 * synchronises `stream` and returns SOBEK_ERR_GRAPH if validation failed.
 */
size_t sobek_graph_prepare_bytes(int64_t N, int64_t E);
int sobek_graph_prepare(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* col,
                        int64_t* src_ptr, int32_t* src_perm, void* ws, size_t ws_bytes,
                        void* stream);

/*
 * sobek_graph_receivers -- fills src_recv[p] = receiver of edge src_perm[p], the column array of the
 * sender-sorted view (it makes that view a plain CSR, so that the source-owned traversal reads its
 * neighbour ids instead of searching row_ptr for them).  Integer work, unique result.  Only enqueues.
 */
int sobek_graph_receivers(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* src_perm,
                          int32_t* src_recv, void* stream);

/*
 * Workspace needed by one call of the given order (0 = fwd, 1 = bwd, 2 = dbwd).  It holds
 * re-laid-out copies of R, the bounded receiver/sender state of one node chunk (at most 2 GiB,
 * whatever the graph), a status word and, for the tensor-core edge kernels, bf16 (hi, lo)
 * copies of the node features they gather from (4 bytes per feature of x, and of gy / vx for
 * orders 1 / 2) and the processing order of the nodes of every chunk (16 bytes per node and graph view).
 * It depends on the plan and on N only -- never on E.
 * The pointer passed as `ws` must be 256-byte aligned.
 */
size_t sobek_workspace_bytes(const sobek_plan* plan, int64_t N, int64_t E, int order);

/* Forward: y (Eqs. receiver_state, receiver_mixing, receiver_matrix_product). */
int sobek_conv_fwd(const sobek_plan* plan, const sobek_graph* g,
                   const float* x, const float* Y, const float* phi, const float* R,
                   float* y, void* ws, size_t ws_bytes, void* stream);

/* First backward: adjoints of (x, Y, phi, R) for the output adjoint gy
 * (Eqs. streamed_radial_adjoints, streamed_operand_adjoints, receiver_adjoint). */
int sobek_conv_bwd(const sobek_plan* plan, const sobek_graph* g,
                   const float* x, const float* Y, const float* phi, const float* R,
                   const float* gy,
                   float* gx, float* gY, float* gphi, float* gR,
                   void* ws, size_t ws_bytes, void* stream);

/*
 * Retaining the receiver state from the forward for the backward (Section "Runtime scratch-budget policy": a
 * forward-retained primal state is reused when it covers all groups and all receivers in one chunk).
 * sobek_conv_fwd_retain is sobek_conv_fwd on a workspace of at least sobek_workspace_bytes(plan, N, E, 1) bytes, laid
 * out as the backward lays it out; it sets *retained to 1 when the state Z of every receiver is left in `ws` (all
 * nodes fit one chunk of the scratch budget and the state schedule is in use), else to 0.
 * sobek_conv_bwd_retained is sobek_conv_bwd with that value passed back: with retained = 1 the caller asserts that
 * `ws` has not been used since by any other call and that plan, graph, x, Y and phi are the ones of the retaining
 * forward; the backward then computes gR from the state in place instead of streaming the edges again.  The call
 * itself consumes the state (one backward per retaining forward).  Results are bitwise those of sobek_conv_bwd.
 * With retained = 0 the two calls are sobek_conv_fwd / sobek_conv_bwd.  Errors: as for those, INVALID_ARG for a
 * null `retained`.
 */
int sobek_conv_fwd_retain(const sobek_plan* plan, const sobek_graph* g, const float* x, const float* Y,
                          const float* phi, const float* R, float* y, void* ws, size_t ws_bytes, void* stream,
                          int* retained);
int sobek_conv_bwd_retained(const sobek_plan* plan, const sobek_graph* g, const float* x, const float* Y,
                            const float* phi, const float* R, const float* gy, float* gx, float* gY, float* gphi,
                            float* gR, void* ws, size_t ws_bytes, void* stream, int retained);

/* Double backward (Eqs. streamed_directional_terms .. streamed_operand_second_adjoints,
 * receiver_double_adjoint) with the direction on gy equal to zero: for the backward map
 * b(x,Y,phi,R; gy) = (gx,gY,gphi,gR) and cotangents v = (vx,vY,vphi,vR) it returns
 * ggy = d<v,b>/d gy and h_theta = d<v,b>/d theta for theta in (x,Y,phi,R). */
int sobek_conv_dbwd(const sobek_plan* plan, const sobek_graph* g,
                    const float* x, const float* Y, const float* phi, const float* R,
                    const float* gy,
                    const float* vx, const float* vY, const float* vphi, const float* vR,
                    float* ggy, float* hx, float* hY, float* hphi, float* hR,
                    void* ws, size_t ws_bytes, void* stream);

/*
 * Geometry front end: the edge inputs recomputed from edge vectors inside the edge kernels, and the gradient
 * that reaches the positions.  The graph inputs Y and phi are edge-sized and "any exact execution must either
 * store or recompute them" (Section "Memory cost of edge-conditioned convolution"; Table memory_complexity lists
 * the spherical harmonics as "stored or recomputed").  These entry points recompute them: the caller passes
 * rvec [E][3], r_e = pos[sender(e)] - pos[receiver(e)] in the receiver-sorted edge order, and no array of width
 * dim_sh or K per edge exists anywhere.  The backward returns the adjoint of the edge vectors g_rvec [E][3],
 * from which the forces follow (Eq. energy_force_symmetry; Section "Introduction": energies and forces).
 *   Y_e    real spherical harmonics of r_e / |r_e|, component normalisation (sum_m Y_lm^2 = 2l+1), no
 *          Condon-Shortley sign, index l*l + l + m with the sine branch at negative m: the basis the coupling
 *          tensors of the plan are expressed in.
 *   phi_e  radial basis of |r_e| (the paper fixes none):
 *          SOBEK_BASIS_BESSEL    sqrt(2/r_cut) sin(n pi r / r_cut) / r * u(r / r_cut), n = 1..K, with the polynomial
 *                                envelope u(d) = 1 - (p+1)(p+2)/2 d^p + p(p+2) d^(p+1) - p(p+1)/2 d^(p+2);
 *          SOBEK_BASIS_GAUSSIAN  exp(-(r - mu_q)^2 / (2 s^2)), mu_q = q s, s = r_cut / (K - 1), q = 0..K-1
 *                                (envelope_p is ignored).
 * Every r_e must be non-zero (an edge of length zero has no direction; nothing is checked).
 * Plans: fully connected or channelwise, ir_mul layout, l_max <= 4, the tensor-core edge kernels in use (the
 * default where the profile allows them: K <= 16, multiplicities multiples of 16 up to 128); otherwise UNSUPPORTED.
 * Workspace: sobek_workspace_bytes(plan, N, E, 0) for the forward, (.., 1) for the backward, (.., 2) for the double
 * backward.  Errors as for sobek_conv_fwd / sobek_conv_bwd / sobek_conv_dbwd.
 *
 * sobek_edge_vectors       rvec[e] = pos[col[e]] - pos[receiver(e)]                       (pos [N][3], rvec [E][3])
 * sobek_conv_geo_fwd       y of sobek_conv_fwd with Y, phi computed from rvec
 * sobek_conv_geo_bwd       gx, gR as sobek_conv_bwd; g_rvec[e] = J_Y(r_e)^T gY_e + J_phi(r_e)^T gphi_e.  Any of
 *                          gx, g_rvec, gR may be NULL (gx needs the sender view of the graph)
 * sobek_conv_geo_dbwd      double backward for a loss on the forces: with cotangents (vx, v_rvec, vR) on the outputs
 *                          (gx, g_rvec, gR) of sobek_conv_geo_bwd it returns ggy = d<v,b>/d gy, hx = d<v,b>/dx and
 *                          hR = d<v,b>/dR (Eqs. streamed_directional_terms .. streamed_operand_second_adjoints with
 *                          the directions vY = J_Y v_rvec, vphi = J_phi v_rvec, which the dual stream passes compute
 *                          from rvec and v_rvec themselves).  Any of the cotangents and of the outputs may be NULL.  The
 *                          derivative with respect to rvec itself is what sobek_conv_geo_dbwd_full adds.
 * sobek_conv_geo_dbwd_full the same three outputs plus h_rvec [E][3] = d<v,b>/d rvec (second derivatives of both
 *                          bases): h_rvec_e = J_Y^T hY_e + J_phi^T hphi_e + d/dr [<J_Y(r) v_e, gY_e> + <J_phi(r) v_e,
 *                          gphi_e>] with the first- and second-order edge adjoints of the convolution.  NOT streaming
 *                          in the edge inputs: Y, phi, their directions and the four edge adjoints are materialised in
 *                          the workspace (8 arrays of E x dim_sh or E x K floats) around stored-input calls of
 *                          sobek_conv_bwd and sobek_conv_dbwd, so every plan those accept is accepted (l_max <= 4,
 *                          K <= 32; else UNSUPPORTED).  Workspace: sobek_geo_dbwd_full_workspace_bytes(plan, N, E).
 *                          Any of vx, v_rvec, vR and of the four outputs may be NULL.
 * sobek_position_gradient  gpos[n] = sum_{e: sender(e) = n} g_rvec[e] - sum_{e: receiver(e) = n} g_rvec[e], the
 *                          adjoint of sobek_edge_vectors (forces are its negative); each node sums its own edges in
 *                          a fixed order (needs src_ptr and src_perm).  Only enqueues.
 */
#define SOBEK_BASIS_BESSEL 0
#define SOBEK_BASIS_GAUSSIAN 1
int sobek_edge_vectors(const sobek_graph* g, const float* pos, float* rvec, void* stream);
int sobek_conv_geo_fwd(const sobek_plan* plan, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                       int envelope_p, const float* x, const float* R, float* y, void* ws, size_t ws_bytes,
                       void* stream);
int sobek_conv_geo_bwd(const sobek_plan* plan, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                       int envelope_p, const float* x, const float* R, const float* gy, float* gx, float* g_rvec,
                       float* gR, void* ws, size_t ws_bytes, void* stream);
int sobek_conv_geo_dbwd(const sobek_plan* plan, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                        int envelope_p, const float* x, const float* R, const float* gy, const float* vx,
                        const float* v_rvec, const float* vR, float* ggy, float* hx, float* hR, void* ws,
                        size_t ws_bytes, void* stream);
size_t sobek_geo_dbwd_full_workspace_bytes(const sobek_plan* plan, int64_t N, int64_t E);
int sobek_conv_geo_dbwd_full(const sobek_plan* plan, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                             int envelope_p, const float* x, const float* R, const float* gy, const float* vx,
                             const float* v_rvec, const float* vR, float* ggy, float* hx, float* hR, float* h_rvec,
                             void* ws, size_t ws_bytes, void* stream);
int sobek_position_gradient(const sobek_graph* g, const float* g_rvec, float* gpos, void* stream);

/*
 * sobek_conv_fwd_static -- the forward convolution with NO workspace argument and no
 * allocation of any kind (the paper has no counterpart; it exists for hosts of this library
 * that cannot allocate device memory when they run the operator: code running inside another
 * framework's fixed memory plan, real-time loops, processes whose device memory was handed out
 * completely at start-up).  Same inputs and output as sobek_conv_fwd, and the same results within the stated
 * tolerance (this path always uses the FP32-pipe edge stream and three-pass GEMMs; SOBEK_FLAG_FAST_GEMM is not
 * honoured; fully connected mode and ir_mul layout only, else UNSUPPORTED).  The scratch that
 * sobek_conv_fwd takes from the caller lives in a fixed array inside the library image:
 * sobek_static_scratch_bytes() bytes (32 MiB) on every GPU that loads the library, held until the
 * process exits.  The call makes no cudaMalloc / cudaFree and calls no allocating routine.
 *   - Limit: about 4*K*N_w + 4*K*F bytes (plus padding) must fit in the array, K*F being
 *     sobek_info.state_floats_fwd (the state of a single node); otherwise SOBEK_ERR_WORKSPACE is
 *     returned and nothing is launched.  Larger graphs only mean more node chunks.
 *   - The first call on a device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - Every call on a device shares the one array, and the array keeps the previous call's
 *     contents: the call clears what must start at zero itself, but two calls whose kernels
 *     overlap on the GPU (different streams) race.  Serialise them.
 *   - The plan must have been created on the device that is current at the call (else INVALID_ARG).
 *   - sobek_static_last_status synchronises `stream` and returns the status word that the kernels of the last
 *     sobek_conv_fwd_static call on the current device left in the array (0, SOBEK_ERR_DEVICE_TIMEOUT,
 *     SOBEK_ERR_GRAPH); CUDA if no such call has been made on this device.
 */
size_t sobek_static_scratch_bytes(void);
int sobek_static_last_status(void* stream);
int sobek_conv_fwd_static(const sobek_plan* plan, const sobek_graph* g,
                          const float* x, const float* Y, const float* phi, const float* R,
                          float* y, void* stream);

/* Self-test of the bounded device-side waits: enqueues a one-thread kernel that waits on a barrier nothing ever
 * completes.  The wait gives up after `limit_ms` (1..2000) milliseconds, writes SOBEK_ERR_DEVICE_TIMEOUT into the
 * status word at the start of `ws` (at least 256 bytes, 256-byte aligned) and the kernel returns normally: the
 * same code path every mbarrier wait of the tensor-core kernels takes if its partner never arrives.  Read the
 * result with sobek_last_device_status.  Errors: INVALID_ARG, CUDA. */
int sobek_selftest_wait_timeout(void* ws, unsigned limit_ms, void* stream);

/* Synchronises `stream`, then returns the status word the kernels of earlier calls wrote
 * into `ws`: 0, SOBEK_ERR_DEVICE_TIMEOUT (a bounded wait gave up), or SOBEK_ERR_GRAPH: a segment bound or an
 * id that a kernel read from row_ptr / col / src_ptr / src_perm / src_recv was out of range.  Such a value is
 * never used as an index (the edge is skipped or reads row 0 instead), so the outputs are finite but wrong. */
int sobek_last_device_status(void* ws, void* stream);

const char* sobek_status_string(int status);

/* Number of kernels this library has launched in this process (for benchmarks). */
int64_t sobek_launch_count(void);

/*
 * Instrumentation for benchmarks (the paper has no counterpart).  While enabled, every kernel
 * launch is bracketed by two CUDA events on its stream.  sobek_timing_collect waits for them,
 * returns per kernel class the summed device time in milliseconds and the number of launches
 * (arrays of sobek_timing_classes() entries), and forgets them.  While enabled, kernels that normally run
 * concurrently on the library's internal side streams are serialised on the caller's stream, so that the
 * brackets do not overlap.  Host-side only; not thread-safe.
 */
int sobek_timing_enable(int on);
int sobek_timing_classes(void);
const char* sobek_timing_class_name(int cls);
int sobek_timing_collect(double* total_ms, int64_t* launches);

/*
 * Measures the sustained FP32 multiply-add rate of the current device (instrumentation for the roofline of the
 * edge kernels; the paper has no counterpart): launches a kernel of independent fused multiply-add chains over and
 * over for about `seconds` (0 < seconds <= 10) of device time, times it with CUDA events and writes the rate in
 * TFLOP/s (2 flops per multiply-add) to *tflops (host).  `scratch` is a device buffer of at least
 * 8192 * (number of SMs) floats that the kernel writes.  Synchronises `stream`.  Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
int sobek_measure_fp32_peak(double seconds, float* scratch, size_t scratch_floats, double* tflops, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SOBEK_H_ */
