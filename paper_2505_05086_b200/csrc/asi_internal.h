// Internal declarations shared by the translation units of the ASI library.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "asi.h"

struct asi_plan;

namespace asi {

// Mode-m view of a contiguous tensor: element (o, k, i) at o*a*I + k*I + i.
// Fibers of the mode are indexed by the flat column q = o*I + i.
struct ModeView {
  int64_t O, a, I, Q;   // Q = O*I = b_m
  int r;
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr int kStatusBytes = 1024;    // status word (int 0), completion counters (ints 16..255)
constexpr int kQRRows = 64;          // rows per CTA in the orthonormalisation kernels
constexpr int kQRMaxRank = 64;       // ranks the register-resident Cholesky-QR kernels cover (above: k_qrb_*)
constexpr int kExpandKC = 32;        // rows of P per CTA in the expand kernel

// Y(o, j, i) = sum_k X(o, k, i) * B(k, j): the small-mode contraction that serves the
// projection V = A_m^T U, the core products, Z1, Z3, and the final expansions.
struct ModeProdArgs {
  const void* X;
  const float* B;
  float* Y;
  int64_t O, a, I, Q;
  int n_out;
  int64_t ldb_k, ldb_j;    // B(k, j) = B[k*ldb_k + j*ldb_j]
  int64_t so, sj, si;      // Y(o, j, i) = Y[o*so + j*sj + i*si]
  void* tc_scratch = nullptr;      // device scratch for the tensor-core kernel's bf16 operand (optional)
  size_t tc_scratch_bytes = 0;
  int* status = nullptr;           // status word of the caller's workspace (a tensor-core wait that expires lands there)
};

// Pp[s](k, j) = sum_{q in split s} X(k, q) * V[q*r + j]
struct ExpandArgs {
  const void* X;
  const float* V;
  float* Pp;
  int64_t O, a, I, Q;
  int r, nsplit;
  int64_t q_per_split;
  void* tc_scratch = nullptr;      // device scratch for the tensor-core kernel's bf16 operand (optional)
  size_t tc_scratch_bytes = 0;
  int* status = nullptr;           // status word of the caller's workspace
};

// One mode's P = A_m (A_m^T U) in a single pass (k_fiber); Pp: [grid][a][r] partials.
struct FiberArgs {
  const void* X;
  const float* U;
  float* Pp;
  int64_t O, a, I, n_tiles;
  int r, vec4;
};

// Modes 3 and 4 of a conv activation in one pass over whole planes (k_plane).
struct PlaneArgs {
  const void* X;
  const float* U3;
  const float* U4;
  float* Pp3;          // [grid][S][r3]
  float* Pp4;          // [grid][S][r4]
  int64_t n_planes;
  int S, r3, r4, vec4;
  int* status = nullptr;   // status word of the workspace (k_plane2: an expired wait on the bulk copy)
};

// One mode with strided fibers, a <= 128, r <= 4 (k_fiber2): both products in one pass, or with
// project_only the mode product Y[o][j][i] = sum_k X[o][k][i] U[k][j] alone.
struct Fiber2Args {
  const void* X;
  const float* U;      // U[k * ldu + j]
  float* Pp;           // [grid][a][r] partials of P (not project_only)
  float* Y;            // project_only: Y[o * y_so + j * y_sj + i]
  int64_t y_so, y_sj;
  int64_t O, I, n_tiles;
  int ldu, a, r, project_only, nstage;
};

struct QRMode {
  const float* Pp;     // [nsplit][a][r]
  double* Pred;        // [a][r]
  double* Gp;          // [nchunk][r][r]
  float* Uout;         // [a][r]
  int a, r, nsplit, nchunk;
};
struct QRArgs {
  QRMode m[ASI_MAX_MODES];
  int* status;
  int gsum;            // set by launch_qr: share 0 of Gp holds the whole of G (else k_qr_solve sums the shares)
};

// Z4[c', j, kh, kw] = sum_{i,h',w'} Z1[i,c',h',w'] Z3pad[i,j,h's+kh-p,w's+kw-p], then
// dW[c', cl, kh, kw] = sum_j Z4[c', j, kh, kw] U2[(g*cg + cl), j].
struct ConvTailArgs {
  const float* Z1;     // [r1][Cout][Ho][Wo]
  const float* Z3;     // [r1][r2][H][W]
  const float* U2;     // [C][r2]
  float* dW;           // [Cout][C/groups][kh][kw]
  int r1, r2, C, Cout, H, W, Ho, Wo, kh, kw, sh, sw, ph, pw, groups;
};

// Fused small-map conv kernels (asi_smallmap_kernels.cu)
constexpr int kRedRows = 8;          // rows of P per CTA in the partial-reduction kernel
struct SmPass1Args {
  const void* act;
  const float* U_prev;
  float* Pp[ASI_MAX_MODES];     // per-mode partials [nsplit][a_m][r_m]
  int* status;                  // status word (int 0) and completion counters (ints 16..255) of the workspace
  int64_t u_off[ASI_MAX_MODES];
  int r[ASI_MAX_MODES];
  int B, C, n_tiles_b;
  unsigned long long wait_ns;   // limit of the bounded wait on the bulk-copy barrier
  int stall_copy;               // test hook: the producer arms the barrier but issues no copy (the wait must expire)
};
// Fixed-order fp64 reduction of the per-tile partials of every P_m, plus per-chunk shares of
// G_m = P_m^T P_m.
struct SmReduceMode {
  const float* Pp;     // [nsplit][a][r], or [nsplit][a][a] Gram matrices A_m A_m^T when gram != 0
  double* Pred;        // [a][r], or [a][a] (the summed Gram matrix) when gram != 0
  double* Gp;          // [nchunk][r][r]
  double* Pg;          // gram != 0 and factor != 0: [a][r], P_m = G_m U_m^prev
  const float* U_prev; // gram != 0 and factor != 0: U_m^prev [a][r]
  int a, r, nsplit, nchunk, gram;
};
constexpr int kRfStride = 80;   // doubles per mode in Rf: rows of R_m at pitch 8, then 1 / diag(R_m) at [64..72)
struct SmReduceArgs {
  SmReduceMode m[ASI_MAX_MODES];
  int factor;          // != 0: the last CTA of each mode factors G_m = R_m^T R_m into Rf (ranks <= 8)
  double* Rf;          // [modes][kRfStride]
  int* counter;        // one per mode, zero on entry, zero again on exit
  int* status;
};
// Finishes Orthogonalize (U_m = P_m R_m^{-1}, rows it needs) in its prologue, then the core.
struct SmCoreArgs {
  const void* act;
  const double* Pred[ASI_MAX_MODES];   // P_m [a][r] in fp64
  const double* Rf;                    // [4][kRfStride]: the Cholesky factors written by the reduction kernel
  float* U_new;
  float* Tp;                    // [n_tiles][core_elems] per-tile partial cores
  float* Tg;                    // [ceil(n_tiles / gs)][core_elems] per-group partial cores
  float* core;
  int* status;
  int* counter;                 // zero on entry, zero again on exit
  int* gcount;                  // one counter per group of gs tiles, same convention
  int gs;
  int64_t u_off[ASI_MAX_MODES];
  int r[ASI_MAX_MODES];
  int B, C, n_tiles;
};
struct SmWgradArgs {
  const float* core;
  const float* U;
  const void* dY;
  float* dW;
  int* status;
  int64_t u_off[ASI_MAX_MODES];
  int r[ASI_MAX_MODES];
  int B, C, Cout, H, W, Ho, Wo, kh, kw, sh, sw, ph, pw, groups, cpb;
  int pj;                       // row pitch (floats) of the staged dY tile
  int bulk;                     // 1: rows staged by 16-byte asynchronous copies (fp32, 16-byte aligned rows)
  int ncl;                      // output channels expanded per round of term 5 (divides cpb)
  int bulk_store;               // 1: dW row blocks leave through the bulk-copy engine (16-byte sized and aligned)
};
size_t sm_pass1_smem(int S, int R, int B, int C);
int sm_pass1_role_c_ctas(int S, int B);
size_t sm_core_smem(int S, int R, int B);
int sm_core_max_rows();
size_t sm_wgrad_smem(const SmWgradArgs& p, int R);
int sm_wgrad_pitch(int J);
cudaError_t launch_sm_pass1(const SmPass1Args& p, int S, int R, bool bf16, cudaStream_t st);
// Tensor-core last-mode product of a bf16 tensor (tcgen05); cudaErrorNotSupported when the shape does not fit.
cudaError_t launch_tc_lastmode(const ModeProdArgs& p, void* scratch, size_t scratch_bytes, cudaStream_t st);
size_t tc_scratch_bytes(int64_t K, int N);
cudaError_t launch_tc_expand(const ExpandArgs& e, void* scratch, size_t scratch_bytes, cudaStream_t st);
cudaError_t launch_sm_reduce(const SmReduceArgs& p, int nd, int max_chunks, cudaStream_t st);
cudaError_t launch_sm_core(const SmCoreArgs& p, int S, int R, bool bf16, cudaStream_t st);
cudaError_t launch_sm_wgrad(const SmWgradArgs& p, int R, bool bf16, cudaStream_t st);
// the same kernels over several layers of one variant in one launch each (n <= sm_max_batch())
int sm_max_batch();
cudaError_t launch_sm_pass1_batched(const SmPass1Args* a, int n, int S, int R, bool bf16, cudaStream_t st);
cudaError_t launch_sm_reduce_batched(const SmReduceArgs* a, const int* max_chunks, int n, cudaStream_t st);
cudaError_t launch_sm_core_batched(const SmCoreArgs* a, int n, int S, int R, bool bf16, cudaStream_t st);
cudaError_t launch_sm_wgrad_batched(const SmWgradArgs* a, int n, int R, bool bf16, cudaStream_t st);

// Benchmark timing aid (asi_profile_begin / asi_profile_end).
struct ProfState {
  int id;
  cudaEvent_t* ev;
  int n_pairs, used;
  double bytes;
};
extern ProfState g_prof;
struct ProfScope {
  cudaStream_t st;
  int slot;
  ProfScope(int id, cudaStream_t s, double alg_bytes) : st(s), slot(-1) {
    if (g_prof.id == id) {
      g_prof.bytes += alg_bytes;
      if (g_prof.used < g_prof.n_pairs) {
        slot = g_prof.used;
        cudaEventRecord(g_prof.ev[2 * slot], st);
      }
      ++g_prof.used;
    }
  }
  ~ProfScope() {
    if (slot >= 0) cudaEventRecord(g_prof.ev[2 * slot + 1], st);
  }
};

// Opt-in to more than 48 KB of dynamic shared memory.  The attribute belongs to a (device, kernel) pair,
// so the sizes already granted are remembered per device.
cudaError_t opt_in_smem(const void* kernel, size_t need);

cudaError_t launch_modeprod(const ModeProdArgs& p, bool x_bf16, cudaStream_t st);
cudaError_t launch_expand(const ExpandArgs& p, bool x_bf16, cudaStream_t st);
cudaError_t launch_qr(const QRArgs& p, int nd, int max_chunks, cudaStream_t st);
cudaError_t launch_qr_solve(const QRArgs& p, int nd, int max_chunks, cudaStream_t st);
cudaError_t launch_fiber(const FiberArgs& p, int grid, bool x_bf16, cudaStream_t st);
size_t fiber_smem(int a);
size_t conv_tail_smem(int r2, int kh, int kw);
cudaError_t launch_plane(const PlaneArgs& p, int grid, bool x_bf16, cudaStream_t st);
size_t plane_smem(int S);
bool fiber2_supported(int64_t O, int64_t a, int64_t I, int r, bool bf16);
int64_t fiber2_tiles(int64_t O, int64_t I);
int fiber2_grid(int64_t O, int64_t a, int64_t I, int r, bool bf16, bool share_sm);
bool fiber_reg_supported(int64_t O, int64_t a, int64_t I, int r, bool bf16);
int fiber_reg_grid(int64_t O, int64_t a, int64_t I, int r, bool bf16);
cudaError_t launch_fiber_reg(const Fiber2Args& p, int grid, bool bf16, cudaStream_t st);
cudaError_t launch_fiber2(const Fiber2Args& p, int grid, bool bf16, cudaStream_t st);
// core = T x_2 U_2^T x_3 U_3^T x_4 U_4^T for T [r1][C][H][W] in one launch (k_core_tail)
struct CoreTailArgs {
  const float* T;
  const float *U2, *U3, *U4;
  float* part;         // [r1][chunks x splits][r2 r3 r4] partial cores
  float* core;
  int* counter;        // zero on entry, zero again on exit
  int r1, r2, r3, r4, C, H, W, RH, cper;
};
bool core_tail_supported(int r2, int r3, int r4, int H, int W);
size_t core_tail_part_elems(int r1, int r2, int r3, int r4, int C, int H, int W);
cudaError_t launch_core_tail(const CoreTailArgs& p, cudaStream_t st);
cudaError_t launch_z3(const float* core, const float* U3, const float* U4, float* Z3, int r12, int r3, int r4,
                      int H, int W, cudaStream_t st);
// token path (asi_token_kernels.cu)
struct LinTailArgs {
  const float* Z;      // Z(l1, l2, o) = Z[l1 * s1 + l2 * s2 + o * so]
  const float* core;   // [L1 L2][r]
  const float* U;      // [Din][r]
  float* dW;           // [Dout][Din]
  float* Z4p;          // [nsplit][Dout][r] shares of Z4 (scratch)
  int nsplit;
  int64_t s1, s2, so;
  int L1, L2, Dout, Din, r;
  int lead_fastest;    // 1: the lead index is the contiguous one in memory (s2 == 1), else o is
};
bool lin_tail_supported(int r);
int lin_tail_nsplit(int nlead, int64_t Dout);
cudaError_t launch_lin_tail(const LinTailArgs& p, cudaStream_t st);
bool modeprod_stage_fits(const ModeProdArgs& p, int* ichunk, size_t* smem);
int modeprod_stage_ksp(int64_t a);
cudaError_t launch_modeprod_stage(const ModeProdArgs& p, int ichunk, size_t smem, cudaStream_t st);
bool plane2_supported(int S, int64_t n_planes, int r3, int r4);
int plane2_grid(int S, int64_t n_planes, int max_ctas);
cudaError_t launch_plane2(const PlaneArgs& p, int grid, bool bf16, cudaStream_t st);
int64_t fiber_tiles(int64_t O, int64_t a, int64_t I);
cudaError_t launch_conv_tail(const ConvTailArgs& p, cudaStream_t st);
cudaError_t launch_conv_tail_split(const ConvTailArgs& p, float* Z4p, int nsp, cudaStream_t st);


}  // namespace asi

namespace asi {
// rank selection aids (asi_spectrum_kernels.cu)
size_t spectrum_ws_bytes(const struct ::asi_plan* pl);
cudaError_t launch_philox_words(uint64_t seed, uint32_t stream, int64_t n_groups, uint32_t* out, cudaStream_t st);
cudaError_t launch_fill_gaussian(uint64_t seed, uint32_t stream, int64_t n, float* out, cudaStream_t st);
cudaError_t launch_mode_spectrum(const struct ::asi_plan* pl, const void* act, double* eig, double* energy, char* w,
                                 cudaStream_t st);
cudaError_t launch_pick_ranks(const struct ::asi_plan* pl, const double* eig, const double* energy, double eps,
                              int r_max, int* ranks, cudaStream_t st);
size_t perplexity_ws_bytes();
cudaError_t launch_perplexity(const float* x, const float* y, int64_t n, double* out, double* part, cudaStream_t st);
}  // namespace asi

struct asi_plan {
  asi_layer_desc_t d;
  int nd;
  int64_t dims[ASI_MAX_MODES];
  int r[ASI_MAX_MODES];
  int64_t N;
  int64_t u_off[ASI_MAX_MODES], u_elems, core_elems;
  int64_t dy_elems, dw_elems, Ho, Wo;
  asi::ModeView mv[ASI_MAX_MODES];
  bool bf16;

  // compress workspace (byte offsets)
  size_t off_V, off_Pp[ASI_MAX_MODES], off_Pred[ASI_MAX_MODES], off_Gp[ASI_MAX_MODES], off_T[2];
  size_t off_Rf, off_Pg[ASI_MAX_MODES];
  size_t off_tc, tc_bytes;         // bf16 operand of the tensor-core products (0 bytes: not used)
  // Token layers run the passes of their modes side by side (they read the same activation and write disjoint
  // scratch): mode m > 0 is enqueued on a stream of the plan's own that forks from and joins the caller's
  // stream by events.  Each mode then has its own V and operand scratch (strides below; 0 when not forked).
  bool fork;
  size_t v_stride, tc_stride;
  struct ForkRes {
    cudaStream_t side[ASI_MAX_MODES - 1];
    cudaEvent_t fork, join[ASI_MAX_MODES - 1];
    int device;
    bool ready, failed;
  };
  mutable ForkRes fr;              // created at the first forked call (under a library-wide lock)
  int tc_mode[ASI_MAX_MODES];      // 0: SIMT, 1: last-mode tensor-core kernels, 2: inner-extent (token) kernels
  int nsplit[ASI_MAX_MODES], nchunk[ASI_MAX_MODES];
  int64_t q_per_split[ASI_MAX_MODES];
  int core_order[ASI_MAX_MODES];
  size_t compress_ws;

  // wgrad workspace (byte offsets)
  size_t off_Z[3], off_Z4p;
  int conv_nsp;                    // > 1: terms 4-5 in two launches with conv_nsp partial Z4 per channel
  bool conv_z3;                    // terms 2-3 in one launch (k_z3)
  int lin_nsplit;                  // shares of the leading indices in the Z4 kernel of the linear backward
  bool lin_reorder;                // linear backward of a bf16 token layer: dY x_2 U_2^T first (tensor cores)
  size_t off_wtc, wtc_bytes;       // bf16 operand scratch of that product
  bool core_tail;                  // the core products after the first in one launch
  size_t off_ctp;                  // partial cores of that launch
  size_t wgrad_ws;

  int launches_compress, launches_wgrad;

  // fused small-map path
  bool fast_compress, fast_wgrad, wgrad_bulk;
  bool small_rank;                 // every rank <= 8: partials are reduced by the parallel fp64 kernel
  bool fiber[ASI_MAX_MODES];       // mode handled by the single-pass fiber kernel
  int fiber_grid[ASI_MAX_MODES];
  bool plane;                      // modes 3 and 4 together by the whole-plane kernel
  int plane_grid;
  bool fiber2[ASI_MAX_MODES];      // ... by its register-tiled successor (ranks <= 4, 16-byte aligned rows)
  bool plane2;                     // 28 x 28 and 56 x 56 planes, ranks <= 4
  int fast_S, fast_R, n_tiles_b, cpb, wgrad_ncl, fold_gs;
};
