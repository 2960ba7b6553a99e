// C ABI of the ASI library: plan construction (host only) and the enqueue sequences.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "asi_internal.h"

using namespace asi;

namespace {

bool valid_ptr(const void* p) { return p != nullptr; }

size_t elem_bytes(const asi_plan* pl) { return pl->bf16 ? 2 : 4; }

void set_mode_views(asi_plan* pl) {
  for (int m = 0; m < pl->nd; ++m) {
    int64_t O = 1, I = 1;
    for (int j = 0; j < m; ++j) O *= pl->dims[j];
    for (int j = m + 1; j < pl->nd; ++j) I *= pl->dims[j];
    pl->mv[m] = ModeView{O, pl->dims[m], I, O * I, pl->r[m]};
  }
}

// dynamic shared memory a fused kernel may ask for: 227 KB per CTA minus up to ~17 KB of static arrays
constexpr size_t kSmemLimit = 208 * 1024;

// Which fused kernels cover this layer (decided once, at plan creation).
void choose_kernels(asi_plan* pl) {
  pl->fast_compress = pl->fast_wgrad = false;
  pl->fast_S = pl->fast_R = pl->n_tiles_b = pl->cpb = 0;
  if (pl->d.kind != ASI_CONV2D || (pl->d.flags & ASI_FLAG_GENERIC_ONLY)) return;
  int rmax = 0;
  for (int m = 0; m < 4; ++m) rmax = std::max(rmax, pl->r[m]);
  if (rmax > 8) return;
  const int R = rmax <= 4 ? 4 : 8;
  pl->fast_R = R;
  const int64_t B = pl->dims[0], C = pl->dims[1], H = pl->dims[2], W = pl->dims[3];
  if (H == W && (H == 7 || H == 14 || H == 16) && B % 8 == 0 && B <= 1024 && C <= 4096 &&
      (H != 7 || C % 4 == 0)) {
    const int S = (int)H;
    if (sm_pass1_smem(S, R, (int)B, (int)C) <= kSmemLimit && sm_core_smem(S, R, (int)B) <= kSmemLimit &&
        B + 4 + 2 * S <= sm_core_max_rows()) {
      pl->fast_compress = true;
      pl->fast_S = S;
      pl->n_tiles_b = (int)((S == 7) ? C / 4 : C);
    }
  }
  if (B <= 4096 && H <= 64 && W <= 64) {
    const int Cout = pl->d.cout;
    const int64_t HoWo = pl->Ho * pl->Wo;
    // channels per CTA: the smallest count that makes a staged row a multiple of 16 bytes (rows can
    // then be staged by 16-byte asynchronous copies); failing that, the smallest that makes it even
    int cpb = 0;
    bool rows_ok = false;
    for (int c = 1; c <= 4 && !cpb; c *= 2)
      if (Cout % c == 0 && (c * HoWo * 4) % 16 == 0) { cpb = c; rows_ok = true; }
    for (int c = 1; c <= 2 && !cpb; c *= 2)
      if (Cout % c == 0 && (c * HoWo) % 2 == 0) cpb = c;
    if (!cpb) return;
    SmWgradArgs a;
    std::memset(&a, 0, sizeof(a));
    for (int m = 0; m < 4; ++m) a.r[m] = pl->r[m];
    a.B = (int)B; a.C = (int)C; a.Cout = Cout; a.H = (int)H; a.W = (int)W;
    a.Ho = (int)pl->Ho; a.Wo = (int)pl->Wo; a.kh = pl->d.kh; a.kw = pl->d.kw; a.cpb = cpb;
    a.ph = pl->d.pad_h; a.pw = pl->d.pad_w; a.groups = pl->d.groups;
    // term 5 expands the channels in two rounds when the staging blocks fit, else one at a time
    a.ncl = cpb >= 2 ? cpb / 2 : 1;
    if (sm_wgrad_smem(a, R) > kSmemLimit) a.ncl = 1;
    if (sm_wgrad_smem(a, R) <= kSmemLimit) {
      pl->fast_wgrad = true;
      pl->cpb = cpb;
      pl->wgrad_ncl = a.ncl;
      pl->wgrad_bulk = rows_ok && !pl->bf16;
    }
  }
}

// Workspace layouts.  Every region is 256-byte aligned; region 0 holds the status word (byte 0)
// and the completion counter of the core kernel (byte 64).
void layout_compress(asi_plan* pl) {
  size_t off = kStatusBytes;
  int rmax = 0;
  for (int m = 0; m < pl->nd; ++m) rmax = std::max(rmax, pl->r[m]);
  pl->small_rank = !pl->fast_compress && rmax <= 8 && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY);
  for (int m = 0; m < ASI_MAX_MODES; ++m) {
    pl->fiber[m] = false;
    pl->fiber_grid[m] = 0;
  }
  pl->plane = false;
  pl->plane_grid = 0;
  if (pl->small_rank && pl->d.kind == ASI_CONV2D && pl->dims[2] == pl->dims[3] && pl->dims[2] % 4 == 0 &&
      pl->dims[2] >= 8 && pl->dims[2] <= 64 && plane_smem((int)pl->dims[2]) <= kSmemLimit) {
    pl->plane = true;
    const int64_t np = 256 / pl->dims[2], planes = pl->dims[0] * pl->dims[1];
    pl->plane_grid = (int)std::min<int64_t>((planes + np - 1) / np, 296);
  }
  // one-pass kernel for every mode with a rank <= 8 and a short fiber, whatever the other modes' ranks
  if (!pl->fast_compress && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY))
    for (int m = 0; m < pl->nd; ++m) {
      if (pl->plane && m >= 2) continue;
      const ModeView& v = pl->mv[m];
      if (pl->r[m] <= 8 && v.a <= 128 && fiber_smem((int)v.a) <= kSmemLimit) {
        pl->fiber[m] = true;
        pl->fiber_grid[m] = (int)std::min<int64_t>(fiber_tiles(v.O, v.a, v.I), 296);
      }
    }
  // register-tiled successors where the shape fits them (one partial per CTA, fewer and larger CTAs)
  pl->plane2 = false;
  for (int m = 0; m < ASI_MAX_MODES; ++m) pl->fiber2[m] = false;
  if (pl->plane && plane2_supported((int)pl->dims[2], pl->dims[0] * pl->dims[1], pl->r[2], pl->r[3])) {
    pl->plane2 = true;
    pl->plane_grid = plane2_grid((int)pl->dims[2], pl->dims[0] * pl->dims[1],
                                 (pl->d.flags & ASI_FLAG_SHARE_SM) ? 148 : 296);
  }
  for (int m = 0; m < pl->nd; ++m)
    if (pl->fiber[m] && fiber2_supported(pl->mv[m].O, pl->mv[m].a, pl->mv[m].I, pl->r[m], pl->bf16)) {
      pl->fiber2[m] = true;
      pl->fiber_grid[m] = fiber2_grid(pl->mv[m].O, pl->mv[m].a, pl->mv[m].I, pl->r[m], pl->bf16,
                                      (pl->d.flags & ASI_FLAG_SHARE_SM) != 0);
    }
  int64_t vmax = 0;
  if (!pl->fast_compress)
    for (int m = 0; m < pl->nd; ++m) vmax = std::max<int64_t>(vmax, pl->mv[m].Q * pl->r[m]);
  pl->fork = pl->d.kind == ASI_LINEAR && pl->nd == 3 && !pl->fast_compress && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY);
  pl->off_V = off;
  pl->v_stride = pl->fork ? align_up((size_t)vmax * 4, 256) : 0;
  off = align_up(off + (size_t)vmax * 4, 256) + (pl->fork ? (size_t)(pl->nd - 1) * pl->v_stride : 0);
  for (int m = 0; m < pl->nd; ++m) {
    const ModeView& v = pl->mv[m];
    const int64_t kchunks = (v.a + kExpandKC - 1) / kExpandKC;
    // about two waves of CTAs, at least four 64-column tiles per split
    int64_t ns = std::max<int64_t>(1, 296 / kchunks);
    ns = std::min<int64_t>(ns, std::max<int64_t>(1, v.Q / 256));
    int64_t qps = (v.Q + ns - 1) / ns;
    qps = (qps + 63) / 64 * 64;
    ns = (v.Q + qps - 1) / qps;
    if (pl->fast_compress) {                                             // one partial per tile; the cold-start
      ns = (m == 1) ? sm_pass1_role_c_ctas(pl->fast_S, (int)pl->dims[0]) : pl->n_tiles_b;   // expansion splits the
      qps = ((v.Q + ns - 1) / ns + 63) / 64 * 64;                        // columns over the same count
    }
    if (pl->fiber[m] || (pl->plane && m >= 2)) {                         // one partial per CTA of k_fiber /
      ns = pl->fiber[m] ? pl->fiber_grid[m] : pl->plane_grid;            // k_plane; the cold-start expansion
      qps = ((v.Q + ns - 1) / ns + 63) / 64 * 64;                        // uses the same count (empty splits
    }                                                                    // write 0)
    pl->nsplit[m] = (int)ns;
    pl->q_per_split[m] = qps;
    const int qr_rows = (pl->fast_compress || pl->small_rank) ? kRedRows : kQRRows;
    pl->nchunk[m] = (int)((v.a + qr_rows - 1) / qr_rows);
    pl->off_Pp[m] = off;
    size_t pp_elems = (size_t)ns * v.a * v.r;
    if (pl->fast_compress && (pl->fast_S == 7 || pl->fast_S == 14) && m >= 2) pp_elems = std::max(pp_elems, (size_t)ns * v.a * v.a);
    off = align_up(off + pp_elems * 4, 256);
    pl->off_Pred[m] = off;
    off = align_up(off + (size_t)v.a * std::max<int64_t>(v.r, (pl->fast_compress && m >= 2) ? v.a : 0) * 8, 256);
    pl->off_Gp[m] = off;
    off = align_up(off + (size_t)pl->nchunk[m] * v.r * v.r * 8, 256);
  }
  // bf16 operand of the tensor-core kernels: products of bf16 tensors with a wide factor (16..64 columns, a
  // multiple of 16) over the last mode (a_m a multiple of 64, >= 128 fibers) or over a mode whose inner
  // extent I is a multiple of 64; the same scratch then serves the mode's expansion (operand = V_m)
  pl->off_tc = off;
  pl->tc_bytes = 0;
  for (int m = 0; m < pl->nd; ++m) pl->tc_mode[m] = 0;
  if (pl->bf16 && !pl->fast_compress)
    for (int m = 0; m < pl->nd; ++m) {
      const ModeView& v = pl->mv[m];
      if (pl->r[m] % 4 != 0 || pl->r[m] < 16 || pl->r[m] > 64) continue;   // factor zero-padded to 16 x
      const bool last = v.I == 1 && v.a % 64 == 0 && v.Q >= 128;
      const bool inner = v.I >= 64 && v.I % 64 == 0 && v.O < 65536;
      if (!last && !inner) continue;
      pl->tc_mode[m] = last ? 1 : 2;
      pl->tc_bytes = std::max(pl->tc_bytes, tc_scratch_bytes(std::max(v.a, v.Q), pl->r[m]));
    }
  pl->tc_stride = pl->fork ? align_up(pl->tc_bytes, 256) : 0;
  off = align_up(off + pl->tc_bytes, 256) + (pl->fork ? (size_t)(pl->nd - 1) * pl->tc_stride : 0);
  pl->off_Rf = off;                                   // Cholesky factors of the fused path
  off = align_up(off + (size_t)ASI_MAX_MODES * kRfStride * 8, 256);
  for (int m = 0; m < ASI_MAX_MODES; ++m) pl->off_Pg[m] = 0;
  if (pl->fast_compress)
    for (int m = 2; m < 4; ++m) {                     // P_m of a Gram mode
      pl->off_Pg[m] = off;
      off = align_up(off + (size_t)pl->dims[m] * pl->r[m] * 8, 256);
    }
  // core chain: contract the mode with the largest a_m / r_m first, then the rest in order
  int order[ASI_MAX_MODES];
  for (int m = 0; m < pl->nd; ++m) order[m] = m;
  int best = 0;
  for (int m = 1; m < pl->nd; ++m)
    if ((double)pl->dims[m] / pl->r[m] > (double)pl->dims[best] / pl->r[best]) best = m;
  std::swap(order[0], order[best]);
  std::sort(order + 1, order + pl->nd);
  std::memcpy(pl->core_order, order, sizeof(order));
  int64_t cd[ASI_MAX_MODES];
  for (int m = 0; m < pl->nd; ++m) cd[m] = pl->dims[m];
  int64_t tmax[2] = {0, 0};
  for (int s = 0; s + 1 < pl->nd; ++s) {
    cd[order[s]] = pl->r[order[s]];
    int64_t n = 1;
    for (int m = 0; m < pl->nd; ++m) n *= cd[m];
    tmax[s & 1] = std::max(tmax[s & 1], n);
  }
  if (pl->fast_compress) {
    tmax[0] = (int64_t)pl->n_tiles_b * pl->core_elems;          // per-tile partial cores
    pl->fold_gs = 8;                                             // tiles per group of the two-level sum
    while ((pl->n_tiles_b + pl->fold_gs - 1) / pl->fold_gs > 192) pl->fold_gs *= 2;
    tmax[1] = (int64_t)((pl->n_tiles_b + pl->fold_gs - 1) / pl->fold_gs) * pl->core_elems;
  }
  for (int t = 0; t < 2; ++t) {
    pl->off_T[t] = off;
    off = align_up(off + (size_t)tmax[t] * 4, 256);
  }
  pl->core_tail = false;
  pl->off_ctp = off;
  if (pl->d.kind == ASI_CONV2D && !pl->fast_compress && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY) &&
      order[0] == 0 && order[1] == 1 && order[2] == 2 && order[3] == 3 &&
      core_tail_supported(pl->r[1], pl->r[2], pl->r[3], (int)pl->dims[2], (int)pl->dims[3])) {
    pl->core_tail = true;
    off = align_up(off + 4 * core_tail_part_elems(pl->r[0], pl->r[1], pl->r[2], pl->r[3], (int)pl->dims[1],
                                                  (int)pl->dims[2], (int)pl->dims[3]), 256);
  }
  pl->compress_ws = off;
  pl->launches_compress = 3;
  if (!pl->fast_compress) {
    pl->launches_compress = 2 + (pl->core_tail ? 2 : pl->nd) + (pl->small_rank ? 0 : 1);   // reduction/QR kernels, core chain
    for (int m = 0; m < pl->nd; ++m)
      pl->launches_compress += (pl->plane && m >= 2) ? (m == 2 ? 1 : 0) : pl->fiber[m] ? 1 : 2;
    // a tensor-core product is two launches (operand split + GEMM): V_m, the expansion when it fits too,
    // and the first core product when it contracts such a mode of the bf16 activation
    for (int m = 0; m < pl->nd; ++m) {
      if (!pl->tc_mode[m]) continue;
      const ModeView& v = pl->mv[m];
      pl->launches_compress += 1;
      if (pl->tc_mode[m] == 2 || (v.a % 8 == 0 && v.a >= 128 && v.Q % 8 == 0)) pl->launches_compress += 1;
      if (pl->core_order[0] == m) pl->launches_compress += 1;
    }
  }
}

void layout_wgrad(asi_plan* pl) {
  size_t off = kStatusBytes;
  int64_t z[3] = {0, 0, 0};
  if (pl->d.kind == ASI_CONV2D) {
    z[0] = (int64_t)pl->r[0] * pl->d.cout * pl->Ho * pl->Wo;          // Z1
    z[1] = (int64_t)pl->r[0] * pl->r[1] * pl->dims[2] * pl->r[3];     // core x_3 U_3
    z[2] = (int64_t)pl->r[0] * pl->r[1] * pl->dims[2] * pl->dims[3];  // Z3
    pl->launches_wgrad = pl->fast_wgrad ? 1 : 4;
  } else {
    const int nlead = pl->nd - 1;
    int64_t rest = pl->d.cout;
    for (int m = 1; m < nlead; ++m) rest *= pl->dims[m];
    z[0] = (int64_t)pl->r[0] * rest;                                   // dY x_1 U_1^T
    z[1] = (nlead > 1) ? (int64_t)pl->r[0] * pl->r[1] * pl->d.cout : 0;  // .. x_2 U_2^T
    pl->lin_nsplit = lin_tail_nsplit(pl->r[0] * (nlead > 1 ? pl->r[1] : 1), pl->d.cout);
    z[2] = (int64_t)pl->lin_nsplit * pl->r[pl->nd - 1] * pl->d.cout;   // Z4 (its shares)
    pl->launches_wgrad = nlead + 2;
    // bf16 token layers whose token-mode factor fits the tensor-core kernel: contract the token mode of dY
    // first (dY is then read once, by tcgen05, and no [r1 x N x Dout] intermediate exists)
    pl->lin_reorder = pl->nd == 3 && pl->bf16 && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY) && pl->r[0] <= 8 &&
                      pl->r[1] % 4 == 0 && pl->r[1] >= 16 && pl->r[1] <= 64 && pl->d.cout % 64 == 0 &&
                      pl->dims[0] < 65536;
    if (pl->lin_reorder) {
      z[0] = pl->dims[0] * pl->d.cout * pl->r[1];                      // dY x_2 U_2^T  [B][Dout][r2]
      z[1] = (int64_t)pl->r[0] * pl->d.cout * pl->r[1];                // .. x_1 U_1^T  [r1][Dout][r2]
      pl->launches_wgrad = 5;
    }
  }
  for (int t = 0; t < 3; ++t) {
    pl->off_Z[t] = off;
    off = align_up(off + (size_t)z[t] * 4, 256);
  }
  pl->off_wtc = off;
  pl->wtc_bytes = 0;
  if (pl->d.kind == ASI_LINEAR && pl->lin_reorder) {
    pl->wtc_bytes = tc_scratch_bytes(pl->dims[1], pl->r[1]);
    off = align_up(off + pl->wtc_bytes, 256);
  }
  pl->conv_nsp = 1;
  pl->off_Z4p = off;
  pl->conv_z3 = pl->d.kind == ASI_CONV2D && !pl->fast_wgrad && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY) &&
                pl->r[2] <= 8 && pl->r[3] <= 8;
  if (pl->conv_z3) pl->launches_wgrad = 3;
  if (pl->d.kind == ASI_CONV2D && !pl->fast_wgrad && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY) &&
      (int64_t)pl->r[0] * pl->Ho * pl->Wo >= 1024 && pl->d.cout < 296) {
    pl->conv_nsp = (int)std::min<int64_t>(16, std::max<int64_t>(2, 592 / pl->d.cout));
    pl->conv_nsp = (int)std::min<int64_t>(pl->conv_nsp, (int64_t)pl->r[0] * pl->Ho);
    off = align_up(off + (size_t)pl->conv_nsp * pl->d.cout * pl->r[1] * pl->d.kh * pl->d.kw * 4, 256);
    pl->launches_wgrad = pl->conv_z3 ? 4 : 5;
  }
  pl->wgrad_ws = off;
}

asi_status_t check_ws(const void* ws, size_t have, size_t need) {
  if (!valid_ptr(ws)) return ASI_ERR_INVALID_ARG;
  if (have < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) return ASI_ERR_WORKSPACE;
  return ASI_OK;
}

thread_local char g_cuda_err[256] = "";

#define ASI_CUDA(call)                                                        \
  do {                                                                        \
    cudaError_t e__ = (call);                                                 \
    if (e__ != cudaSuccess) {                                                 \
      snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", #call, cudaGetErrorString(e__)); \
      return ASI_ERR_CUDA;                                                    \
    }                                                                         \
  } while (0)

// Argument blocks of the fused small-map kernels for one layer (shared by the single-layer and the
// batched entry points).
void build_fused_pass1(const asi_plan* pl, const void* act, const float* U_prev, char* w, SmPass1Args* a) {
  a->act = act;
  a->U_prev = U_prev;
  for (int m = 0; m < 4; ++m) {
    a->Pp[m] = reinterpret_cast<float*>(w + pl->off_Pp[m]);
    a->u_off[m] = pl->u_off[m];
    a->r[m] = pl->r[m];
  }
  a->status = reinterpret_cast<int*>(w);     // cleared by the kernel itself
  a->B = (int)pl->dims[0];
  a->C = (int)pl->dims[1];
  a->n_tiles_b = pl->n_tiles_b;
  a->stall_copy = (pl->d.flags & ASI_FLAG_TEST_EXPIRE_WAIT) ? 1 : 0;
  a->wait_ns = a->stall_copy ? 1000000ull : 1000000000ull;      // 1 ms under the test hook, else 1 s
}

int build_fused_reduce(const asi_plan* pl, char* w, const float* gram_U_prev, SmReduceArgs* ra) {
  int max_chunks = 1;
  std::memset(ra, 0, sizeof(*ra));
  for (int m = 0; m < pl->nd; ++m) {
    ra->m[m].Pp = reinterpret_cast<const float*>(w + pl->off_Pp[m]);
    ra->m[m].Pred = reinterpret_cast<double*>(w + pl->off_Pred[m]);
    ra->m[m].Gp = reinterpret_cast<double*>(w + pl->off_Gp[m]);
    ra->m[m].a = (int)pl->dims[m];
    ra->m[m].r = pl->r[m];
    ra->m[m].nsplit = pl->nsplit[m];
    ra->m[m].nchunk = pl->nchunk[m];
    if (gram_U_prev && (pl->fast_S == 7 || pl->fast_S == 14) && m >= 2) {
      ra->m[m].gram = 1;
      ra->m[m].nchunk = (int)((pl->dims[m] * pl->dims[m] + 24) / 25);   // ~25 Gram elements per CTA
      ra->m[m].Pg = reinterpret_cast<double*>(w + pl->off_Pg[m]);
      ra->m[m].U_prev = gram_U_prev + pl->u_off[m];
    }
    max_chunks = std::max(max_chunks, ra->m[m].nchunk);
  }
  ra->factor = 1;
  ra->Rf = reinterpret_cast<double*>(w + pl->off_Rf);
  ra->counter = reinterpret_cast<int*>(w) + 20;
  ra->status = reinterpret_cast<int*>(w);
  return max_chunks;
}

void build_fused_core(const asi_plan* pl, const void* act, float* U_new, float* core, char* w, bool gram_modes,
                      SmCoreArgs* c) {
  c->act = act;
  c->U_new = U_new;
  c->Rf = reinterpret_cast<const double*>(w + pl->off_Rf);
  c->Tp = reinterpret_cast<float*>(w + pl->off_T[0]);
  c->core = core;
  c->status = reinterpret_cast<int*>(w);
  c->counter = reinterpret_cast<int*>(w) + 16;
  c->gcount = reinterpret_cast<int*>(w) + 64;
  c->gs = pl->fold_gs;
  c->Tg = reinterpret_cast<float*>(w + pl->off_T[1]);
  for (int m = 0; m < 4; ++m) {
    const bool gram = gram_modes && (pl->fast_S == 7 || pl->fast_S == 14) && m >= 2;
    c->Pred[m] = reinterpret_cast<const double*>(w + (gram ? pl->off_Pg[m] : pl->off_Pred[m]));
    c->u_off[m] = pl->u_off[m];
    c->r[m] = pl->r[m];
  }
  c->B = (int)pl->dims[0];
  c->C = (int)pl->dims[1];
  c->n_tiles = pl->n_tiles_b;
}

// false: dY is not aligned as the staged copies of this plan need
bool build_fused_wgrad(const asi_plan* pl, const float* core, const float* U, const void* dY, float* dW, char* w,
                       SmWgradArgs* g) {
  g->core = core; g->U = U; g->dY = dY; g->dW = dW;
  for (int m = 0; m < 4; ++m) {
    g->u_off[m] = pl->u_off[m];
    g->r[m] = pl->r[m];
  }
  g->B = (int)pl->dims[0]; g->C = (int)pl->dims[1]; g->Cout = pl->d.cout;
  g->H = (int)pl->dims[2]; g->W = (int)pl->dims[3]; g->Ho = (int)pl->Ho; g->Wo = (int)pl->Wo;
  g->kh = pl->d.kh; g->kw = pl->d.kw; g->sh = pl->d.stride_h; g->sw = pl->d.stride_w;
  g->ph = pl->d.pad_h; g->pw = pl->d.pad_w; g->groups = pl->d.groups; g->cpb = pl->cpb;
  g->ncl = pl->wgrad_ncl;
  g->pj = sm_wgrad_pitch(pl->cpb * (int)(pl->Ho * pl->Wo));
  g->bulk = pl->wgrad_bulk ? 1 : 0;
  if (g->bulk && (reinterpret_cast<uintptr_t>(dY) & 15u)) return false;
  g->status = reinterpret_cast<int*>(w);
  g->bulk_store = (((pl->dims[1] / pl->d.groups) * pl->d.kh * pl->d.kw) % 4 == 0 &&
                   (reinterpret_cast<uintptr_t>(dW) & 15u) == 0) ? 1 : 0;
  return true;
}

// U_m^{new} = Orthogonalize(P_m) for all modes given the split partials.
// gram_U_prev != nullptr: the partials of modes 3 and 4 of a 7x7 or 14x14 map are Gram matrices A_m A_m^T
// (written by the fused first pass) and P_m = G_m U_m^prev is formed during the reduction.
asi_status_t orthogonalize_all(const asi_plan* pl, float* U_new, char* w, const float* gram_U_prev,
                               cudaStream_t st) {
  int max_chunks = 1;
  for (int m = 0; m < pl->nd; ++m) max_chunks = std::max(max_chunks, pl->nchunk[m]);
  if (pl->fast_compress) {
    SmReduceArgs ra;
    max_chunks = build_fused_reduce(pl, w, gram_U_prev, &ra);
    ASI_CUDA(launch_sm_reduce(ra, pl->nd, max_chunks, st));
    return ASI_OK;      // the core kernel solves for the rows of U_m
  }
  if (pl->small_rank) {
    SmReduceArgs ra;
    std::memset(&ra, 0, sizeof(ra));
    for (int m = 0; m < pl->nd; ++m) {
      ra.m[m].Pp = reinterpret_cast<const float*>(w + pl->off_Pp[m]);
      ra.m[m].Pred = reinterpret_cast<double*>(w + pl->off_Pred[m]);
      ra.m[m].Gp = reinterpret_cast<double*>(w + pl->off_Gp[m]);
      ra.m[m].a = (int)pl->dims[m];
      ra.m[m].r = pl->r[m];
      ra.m[m].nsplit = pl->nsplit[m];
      ra.m[m].nchunk = pl->nchunk[m];
    }
    ASI_CUDA(launch_sm_reduce(ra, pl->nd, max_chunks, st));
  }
  QRArgs qa;
  std::memset(&qa, 0, sizeof(qa));
  for (int m = 0; m < pl->nd; ++m) {
    qa.m[m].Pp = reinterpret_cast<const float*>(w + pl->off_Pp[m]);
    qa.m[m].Pred = reinterpret_cast<double*>(w + pl->off_Pred[m]);
    qa.m[m].Gp = reinterpret_cast<double*>(w + pl->off_Gp[m]);
    qa.m[m].Uout = U_new + pl->u_off[m];
    qa.m[m].a = (int)pl->dims[m];
    qa.m[m].r = pl->r[m];
    qa.m[m].nsplit = pl->nsplit[m];
    qa.m[m].nchunk = pl->nchunk[m];
  }
  qa.status = reinterpret_cast<int*>(w);
  if (pl->small_rank) ASI_CUDA(launch_qr_solve(qa, pl->nd, max_chunks, st));
  else ASI_CUDA(launch_qr(qa, pl->nd, max_chunks, st));
  return ASI_OK;
}

// A mode product that streams a large tensor once: the register-tiled kernel when the shape fits it
// (strided fibers, a <= 128, at most four outputs, contiguous outputs per (o, j)), else the general one.
cudaError_t stream_modeprod(const asi_plan* pl, const ModeProdArgs& a, bool x_bf16, cudaStream_t st) {
  const bool fits = !(pl->d.flags & ASI_FLAG_GENERIC_ONLY) && a.si == 1 && a.ldb_j == 1 && a.sj == a.I &&
                    a.so == (int64_t)a.n_out * a.I && a.Q * a.a >= (1 << 20) &&
                    fiber2_supported(a.O, a.a, a.I, a.n_out, x_bf16) &&
                    (reinterpret_cast<uintptr_t>(a.X) & 15u) == 0 && (reinterpret_cast<uintptr_t>(a.Y) & 15u) == 0;
  if (!fits) {
    int ichunk = 0;
    size_t smem = 0;
    if (!x_bf16 && !(pl->d.flags & ASI_FLAG_GENERIC_ONLY) && modeprod_stage_fits(a, &ichunk, &smem))
      return launch_modeprod_stage(a, ichunk, smem, st);      // few columns, long mode
    return launch_modeprod(a, x_bf16, st);
  }
  Fiber2Args f;
  std::memset(&f, 0, sizeof(f));
  f.X = a.X;
  f.U = a.B;
  f.ldu = (int)a.ldb_k;
  f.Y = a.Y;
  f.y_so = a.so;
  f.y_sj = a.sj;
  f.O = a.O; f.I = a.I; f.a = (int)a.a; f.r = a.n_out;
  f.n_tiles = fiber2_tiles(a.O, a.I);
  f.project_only = 1;
  return launch_fiber2(f, fiber2_grid(a.O, a.a, a.I, a.n_out, x_bf16, (pl->d.flags & ASI_FLAG_SHARE_SM) != 0),
                       x_bf16, st);
}

// Orthogonalize, then core = A x_1 U_1^T ... x_n U_n^T (Algorithm 1, core update with U^T).
asi_status_t finish_compress(const asi_plan* pl, const void* act, float* U_new, float* core,
                             char* w, const float* gram_U_prev, cudaStream_t st) {
  asi_status_t qs = orthogonalize_all(pl, U_new, w, gram_U_prev, st);
  if (qs != ASI_OK) return qs;
  if (pl->fast_compress) {
    SmCoreArgs c;
    build_fused_core(pl, act, U_new, core, w, gram_U_prev != nullptr, &c);
    ASI_CUDA(launch_sm_core(c, pl->fast_S, pl->fast_R, pl->bf16, st));
    return ASI_OK;
  }
  int64_t cd[ASI_MAX_MODES];
  for (int m = 0; m < pl->nd; ++m) cd[m] = pl->dims[m];
  const void* src = act;
  bool src_bf16 = pl->bf16;
  for (int s = 0; s < pl->nd; ++s) {
    const int m = pl->core_order[s];
    ModeProdArgs a;
    a.X = src;
    a.B = U_new + pl->u_off[m];
    a.O = 1;
    a.I = 1;
    for (int j = 0; j < m; ++j) a.O *= cd[j];
    for (int j = m + 1; j < pl->nd; ++j) a.I *= cd[j];
    a.a = cd[m];
    a.Q = a.O * a.I;
    a.n_out = pl->r[m];
    a.ldb_k = pl->r[m];
    a.ldb_j = 1;
    a.so = (int64_t)pl->r[m] * a.I;
    a.sj = a.I;
    a.si = 1;
    float* dst = (s == pl->nd - 1) ? core : reinterpret_cast<float*>(w + pl->off_T[s & 1]);
    a.Y = dst;
    a.tc_scratch = w + pl->off_tc;
    a.tc_scratch_bytes = pl->tc_bytes;
    a.status = reinterpret_cast<int*>(w);
    ASI_CUDA(stream_modeprod(pl, a, src_bf16, st));
    cd[m] = pl->r[m];
    src = dst;
    src_bf16 = false;
    if (s == 0 && pl->core_tail) {
      CoreTailArgs t;
      std::memset(&t, 0, sizeof(t));
      t.T = dst;
      t.U2 = U_new + pl->u_off[1]; t.U3 = U_new + pl->u_off[2]; t.U4 = U_new + pl->u_off[3];
      t.part = reinterpret_cast<float*>(w + pl->off_ctp);
      t.core = core;
      t.counter = reinterpret_cast<int*>(w) + 32;
      t.r1 = pl->r[0]; t.r2 = pl->r[1]; t.r3 = pl->r[2]; t.r4 = pl->r[3];
      t.C = (int)pl->dims[1]; t.H = (int)pl->dims[2]; t.W = (int)pl->dims[3];
      ASI_CUDA(launch_core_tail(t, st));
      break;
    }
  }
  return ASI_OK;
}

std::mutex g_fork_mu;

// The plan's side streams and events, created on first use for the current device.  false: run the modes one
// after another on the caller's stream (creation failed once, or the plan was first used on another device).
bool fork_ready(const asi_plan* pl) {
  if (!pl->fork) return false;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  std::lock_guard<std::mutex> lock(g_fork_mu);
  asi_plan::ForkRes& f = pl->fr;
  if (f.failed) return false;
  if (f.ready) return f.device == dev;
  bool ok = cudaEventCreateWithFlags(&f.fork, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < pl->nd - 1; ++i)
    ok = cudaStreamCreateWithFlags(&f.side[i], cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&f.join[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    (void)cudaGetLastError();
    f.failed = true;
    return false;
  }
  f.device = dev;
  f.ready = true;
  return true;
}

asi_status_t expand_mode(const asi_plan* pl, int m, const void* act, const float* V, char* w,
                         cudaStream_t st, int slot = 0) {
  const ModeView& v = pl->mv[m];
  ExpandArgs e;
  e.X = act;
  e.V = V;
  e.Pp = reinterpret_cast<float*>(w + pl->off_Pp[m]);
  e.O = v.O;
  e.a = v.a;
  e.I = v.I;
  e.Q = v.Q;
  e.r = v.r;
  e.nsplit = pl->nsplit[m];
  e.q_per_split = pl->q_per_split[m];
  e.tc_scratch = w + pl->off_tc + (size_t)slot * pl->tc_stride;
  e.tc_scratch_bytes = pl->tc_bytes;
  e.status = reinterpret_cast<int*>(w);
  ASI_CUDA(launch_expand(e, pl->bf16, st));
  return ASI_OK;
}

}  // namespace

extern "C" {

const char* asi_status_string(asi_status_t s) {
  switch (s) {
    case ASI_OK: return "ok";
    case ASI_ERR_INVALID_ARG: return "invalid argument";
    case ASI_ERR_UNSUPPORTED: return "unsupported configuration";
    case ASI_ERR_RANK_RANGE: return "rank outside [1, min(a_m, b_m)]";
    case ASI_ERR_WORKSPACE: return "workspace too small or misaligned";
    case ASI_ERR_CUDA: return "CUDA runtime error";
    case ASI_ERR_RANK_DEFICIENT: return "rank-deficient subspace iterate";
    case ASI_ERR_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

const char* asi_last_cuda_error(void) { return g_cuda_err; }

asi_status_t asi_plan_create(const asi_layer_desc_t* desc, asi_plan_t** out) {
  if (!desc || !out) return ASI_ERR_INVALID_ARG;
  const asi_layer_desc_t& d = *desc;
  if (d.kind != ASI_CONV2D && d.kind != ASI_LINEAR) return ASI_ERR_INVALID_ARG;
  if (d.in_dtype != ASI_F32 && d.in_dtype != ASI_BF16) return ASI_ERR_INVALID_ARG;
  if (d.kind == ASI_CONV2D && d.ndim != 4) return ASI_ERR_UNSUPPORTED;
  if (d.kind == ASI_LINEAR && d.ndim != 2 && d.ndim != 3) return ASI_ERR_UNSUPPORTED;
  if (d.cout < 1) return ASI_ERR_INVALID_ARG;
  int64_t N = 1;
  for (int m = 0; m < d.ndim; ++m) {
    if (d.dims[m] < 1 || d.dims[m] > (int64_t)1 << 31) return ASI_ERR_INVALID_ARG;
    N *= d.dims[m];
    if (N > (int64_t)1 << 40) return ASI_ERR_UNSUPPORTED;
  }
  for (int m = 0; m < d.ndim; ++m) {
    const int64_t a = d.dims[m], b = N / a;
    if (d.ranks[m] < 1 || d.ranks[m] > std::min(a, b)) return ASI_ERR_RANK_RANGE;
    if (d.ranks[m] > ASI_MAX_RANK) return ASI_ERR_UNSUPPORTED;
  }
  int64_t Ho = 0, Wo = 0;
  if (d.kind == ASI_CONV2D) {
    if (d.kh < 1 || d.kw < 1 || d.stride_h < 1 || d.stride_w < 1 || d.pad_h < 0 || d.pad_w < 0 ||
        d.groups < 1)
      return ASI_ERR_INVALID_ARG;
    if (d.dil_h != 1 || d.dil_w != 1) return ASI_ERR_UNSUPPORTED;
    if (d.dims[1] % d.groups || d.cout % d.groups) return ASI_ERR_INVALID_ARG;
    if (d.kh > 16 || d.kw > 16) return ASI_ERR_UNSUPPORTED;
    const int64_t hn = d.dims[2] + 2 * d.pad_h - d.kh, wn = d.dims[3] + 2 * d.pad_w - d.kw;
    if (hn < 0 || wn < 0) return ASI_ERR_INVALID_ARG;
    Ho = hn / d.stride_h + 1;
    Wo = wn / d.stride_w + 1;
  }
  asi_plan* pl = new (std::nothrow) asi_plan;
  if (!pl) return ASI_ERR_INVALID_ARG;
  std::memset(pl, 0, sizeof(*pl));
  pl->d = d;
  pl->nd = d.ndim;
  pl->N = N;
  pl->bf16 = d.in_dtype == ASI_BF16;
  pl->Ho = Ho;
  pl->Wo = Wo;
  int64_t uo = 0, ce = 1;
  for (int m = 0; m < d.ndim; ++m) {
    pl->dims[m] = d.dims[m];
    pl->r[m] = d.ranks[m];
    pl->u_off[m] = uo;
    uo += d.dims[m] * d.ranks[m];
    ce *= d.ranks[m];
  }
  pl->u_elems = uo;
  pl->core_elems = ce;
  if (d.kind == ASI_CONV2D) {
    pl->dy_elems = d.dims[0] * d.cout * Ho * Wo;
    pl->dw_elems = (int64_t)d.cout * (d.dims[1] / d.groups) * d.kh * d.kw;
  } else {
    pl->dy_elems = N / d.dims[d.ndim - 1] * d.cout;
    pl->dw_elems = (int64_t)d.cout * d.dims[d.ndim - 1];
  }
  set_mode_views(pl);
  choose_kernels(pl);
  layout_compress(pl);
  layout_wgrad(pl);
  *out = pl;
  return ASI_OK;
}

asi_status_t asi_plan_destroy(asi_plan_t* plan) {
  if (!plan) return ASI_ERR_INVALID_ARG;
  if (plan->fr.ready) {
    for (int i = 0; i < plan->nd - 1; ++i) {
      cudaStreamDestroy(plan->fr.side[i]);
      cudaEventDestroy(plan->fr.join[i]);
    }
    cudaEventDestroy(plan->fr.fork);
  }
  delete plan;
  return ASI_OK;
}

asi_status_t asi_plan_query(const asi_plan_t* pl, asi_plan_info_t* info) {
  if (!pl || !info) return ASI_ERR_INVALID_ARG;
  std::memset(info, 0, sizeof(*info));
  info->compress_ws_bytes = pl->compress_ws;
  info->wgrad_ws_bytes = pl->wgrad_ws;
  double sum_r = 0, sum_r3 = 0;
  for (int m = 0; m < pl->nd; ++m) {
    info->u_offset[m] = pl->u_off[m];
    sum_r += pl->r[m];
    sum_r3 += (double)pl->r[m] * pl->r[m] * pl->r[m];
  }
  info->u_elems = pl->u_elems;
  info->core_elems = pl->core_elems;
  info->act_elems = pl->N;
  info->dy_elems = pl->dy_elems;
  info->dw_elems = pl->dw_elems;
  info->out_h = pl->Ho;
  info->out_w = pl->Wo;
  info->compressed_elems = pl->core_elems + pl->u_elems;
  info->ratio_RC = (double)pl->N / (double)info->compressed_elems;
  info->macs_O_ASI = 2.0 * (double)pl->N * sum_r + sum_r3;
  if (pl->d.kind == ASI_CONV2D) {
    const double B = pl->dims[0], C = pl->dims[1], H = pl->dims[2], W = pl->dims[3];
    const double r1 = pl->r[0], r2 = pl->r[1], r3 = pl->r[2], r4 = pl->r[3];
    const double Co = pl->d.cout, HoWo = (double)pl->Ho * pl->Wo, D2 = (double)pl->d.kh * pl->d.kw;
    info->macs_C_ASI = r1 * B * Co * HoWo + r1 * r2 * r3 * r4 * H + r1 * r2 * r4 * H * W +
                       r1 * r2 * Co * HoWo * D2 + r2 * Co * C * D2;
    info->macs_C_vanilla = D2 * C * Co * B * HoWo;
  } else {
    // linear layers (Sec. 3.1 footnote): Z = dY x_1 U_1^T (x_2 U_2^T), Z4 = Z . core over the leading ranks,
    // dW = Z4 U_last^T -- one term per contraction, like the five terms of the conv cost
    const int nd = pl->nd;
    const double Do = pl->d.cout, Din = pl->dims[nd - 1], rl = pl->r[nd - 1];
    double macs = 0.0, lead = 1.0, rest = Do;
    for (int m = 1; m < nd - 1; ++m) rest *= (double)pl->dims[m];
    for (int m = 0; m < nd - 1; ++m) {
      macs += lead * pl->r[m] * (double)pl->dims[m] * rest;      // contract mode m of the running tensor
      lead *= pl->r[m];
      if (m + 1 < nd - 1) rest /= (double)pl->dims[m + 1];
    }
    macs += lead * rl * Do + rl * Do * Din;
    info->macs_C_ASI = macs;
    info->macs_C_vanilla = (double)pl->N * pl->d.cout;
  }
  return ASI_OK;
}

int32_t asi_launch_count(const asi_plan_t* pl, int32_t which) {
  if (!pl) return -1;
  return which == 0 ? pl->launches_compress : pl->launches_wgrad;
}

// allow_fork: the passes of a token layer's modes may run side by side on the plan's own streams
static asi_status_t compress_impl(const asi_plan_t* pl, const void* act, const float* U_prev, float* U_new,
                                  float* core, void* ws, size_t ws_bytes, void* stream, bool allow_fork) {
  if (!pl || !valid_ptr(act) || !valid_ptr(U_prev) || !valid_ptr(U_new) || !valid_ptr(core))
    return ASI_ERR_INVALID_ARG;
  if (U_prev == U_new) return ASI_ERR_INVALID_ARG;
  asi_status_t s = check_ws(ws, ws_bytes, pl->compress_ws);
  if (s != ASI_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if (pl->fast_compress) {
    // fp32 tiles are staged by 16-byte asynchronous copies, which need 16-byte aligned sources
    if (!pl->bf16 && (reinterpret_cast<uintptr_t>(act) & 15u)) return ASI_ERR_INVALID_ARG;
    SmPass1Args a;
    build_fused_pass1(pl, act, U_prev, w, &a);
    ASI_CUDA(launch_sm_pass1(a, pl->fast_S, pl->fast_R, pl->bf16, st));
    return finish_compress(pl, act, U_new, core, w, U_prev, st);
  }
  ASI_CUDA(cudaMemsetAsync(w, 0, kStatusBytes, st));
  float* V = reinterpret_cast<float*>(w + pl->off_V);
  const bool forked = allow_fork && fork_ready(pl);
  if (forked) {
    ASI_CUDA(cudaEventRecord(pl->fr.fork, st));
    for (int i = 0; i < pl->nd - 1; ++i) ASI_CUDA(cudaStreamWaitEvent(pl->fr.side[i], pl->fr.fork, 0));
  }
  const cudaStream_t st0 = st;
  if (pl->plane) {
    PlaneArgs g;
    g.X = act;
    g.U3 = U_prev + pl->u_off[2];
    g.U4 = U_prev + pl->u_off[3];
    g.Pp3 = reinterpret_cast<float*>(w + pl->off_Pp[2]);
    g.Pp4 = reinterpret_cast<float*>(w + pl->off_Pp[3]);
    g.n_planes = pl->dims[0] * pl->dims[1];
    g.S = (int)pl->dims[2];
    g.r3 = pl->r[2];
    g.r4 = pl->r[3];
    g.vec4 = (!pl->bf16 && (reinterpret_cast<uintptr_t>(act) & 15u) == 0) ? 1 : 0;
    g.status = reinterpret_cast<int*>(w);
    if (pl->plane2) {
      if (reinterpret_cast<uintptr_t>(act) & 15u) return ASI_ERR_INVALID_ARG;   // bulk copies need 16-byte alignment
      ASI_CUDA(launch_plane2(g, pl->plane_grid, pl->bf16, st));
    } else {
      ASI_CUDA(launch_plane(g, pl->plane_grid, pl->bf16, st));
    }
  }
  for (int m = 0; m < pl->nd; ++m)                   // argument errors before anything is forked
    if (pl->fiber2[m] && !(pl->plane && m >= 2) && (reinterpret_cast<uintptr_t>(act) & 15u)) return ASI_ERR_INVALID_ARG;
  for (int m = 0; m < pl->nd; ++m) {
    const ModeView& v = pl->mv[m];
    if (pl->plane && m >= 2) continue;
    const int slot = forked ? m : 0;                 // scratch and stream of this mode's pass
    st = (forked && m > 0) ? pl->fr.side[m - 1] : st0;
    V = reinterpret_cast<float*>(w + pl->off_V + (size_t)slot * pl->v_stride);
    if (pl->fiber2[m]) {
      if (reinterpret_cast<uintptr_t>(act) & 15u) return ASI_ERR_INVALID_ARG;
      Fiber2Args f;
      std::memset(&f, 0, sizeof(f));
      f.X = act;
      f.U = U_prev + pl->u_off[m];
      f.ldu = v.r;
      f.Pp = reinterpret_cast<float*>(w + pl->off_Pp[m]);
      f.O = v.O; f.I = v.I; f.a = (int)v.a; f.r = v.r;
      f.n_tiles = fiber2_tiles(v.O, v.I);
      ASI_CUDA(launch_fiber2(f, pl->fiber_grid[m], pl->bf16, st));
      continue;
    }
    if (pl->fiber[m]) {
      // both products of the mode in one pass; V stays on chip
      FiberArgs f;
      f.X = act;
      f.U = U_prev + pl->u_off[m];
      f.Pp = reinterpret_cast<float*>(w + pl->off_Pp[m]);
      f.O = v.O; f.a = v.a; f.I = v.I;
      f.n_tiles = fiber_tiles(v.O, v.a, v.I);
      f.r = v.r;
      f.vec4 = (!pl->bf16 && v.I % 4 == 0 && (reinterpret_cast<uintptr_t>(act) & 15u) == 0) ? 1 : 0;
      ASI_CUDA(launch_fiber(f, pl->fiber_grid[m], pl->bf16, st));
      continue;
    }
    // V = A_m^T U_m^{prev}, stored [b_m x r_m]
    ModeProdArgs a;
    a.X = act;
    a.B = U_prev + pl->u_off[m];
    a.Y = V;
    a.O = v.O;
    a.a = v.a;
    a.I = v.I;
    a.Q = v.Q;
    a.n_out = v.r;
    a.ldb_k = v.r;
    a.ldb_j = 1;
    a.so = v.I * v.r;
    a.sj = 1;
    a.si = v.r;
    a.tc_scratch = w + pl->off_tc + (size_t)slot * pl->tc_stride;
    a.tc_scratch_bytes = pl->tc_bytes;
    a.status = reinterpret_cast<int*>(w);
    ASI_CUDA(launch_modeprod(a, pl->bf16, st));
    // P = A_m V
    s = expand_mode(pl, m, act, V, w, st, slot);
    if (s != ASI_OK) return s;
  }
  st = st0;
  if (forked)
    for (int i = 0; i < pl->nd - 1; ++i) {
      ASI_CUDA(cudaEventRecord(pl->fr.join[i], pl->fr.side[i]));
      ASI_CUDA(cudaStreamWaitEvent(st, pl->fr.join[i], 0));
    }
  return finish_compress(pl, act, U_new, core, w, nullptr, st);
}

asi_status_t asi_compress(const asi_plan_t* pl, const void* act, const float* U_prev, float* U_new,
                          float* core, void* ws, size_t ws_bytes, void* stream) {
  return compress_impl(pl, act, U_prev, U_new, core, ws, ws_bytes, stream, true);
}

// ---------------------------------------------------------------------------------------------
// Batched entry points: the layers a training step compresses together (Algorithm 1 runs once per
// fine-tuned layer and step; Sec. 4 fine-tunes the last 2..4 layers).  Layers on the fused small-map path
// that share a kernel variant go through ONE launch of each kernel stage, their argument blocks in a
// table the CTAs index; the remaining layers are enqueued one after another on the same stream.
// ---------------------------------------------------------------------------------------------
namespace {
struct Variant {
  int S, R, bf16;
  bool operator==(const Variant& o) const { return S == o.S && R == o.R && bf16 == o.bf16; }
};
}  // namespace

asi_status_t asi_compress_batched(const asi_plan_t* const* plans, const void* const* acts,
                                  const float* const* U_prev, float* const* U_new, float* const* cores,
                                  void* const* ws, const size_t* ws_bytes, int32_t n, void* stream) {
  if (!plans || !acts || !U_prev || !U_new || !cores || !ws || !ws_bytes || n < 1 || n > 4096)
    return ASI_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    const asi_plan* pl = plans[i];
    if (!pl || !valid_ptr(acts[i]) || !valid_ptr(U_prev[i]) || !valid_ptr(U_new[i]) || !valid_ptr(cores[i]))
      return ASI_ERR_INVALID_ARG;
    if (U_prev[i] == U_new[i]) return ASI_ERR_INVALID_ARG;
    const asi_status_t s = check_ws(ws[i], ws_bytes[i], pl->compress_ws);
    if (s != ASI_OK) return s;
    if (pl->fast_compress && !pl->bf16 && (reinterpret_cast<uintptr_t>(acts[i]) & 15u)) return ASI_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (ws[j] == ws[i]) return ASI_ERR_INVALID_ARG;            // every layer needs a workspace of its own
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::vector<char> done(n, 0);
  const int maxb = sm_max_batch();
  for (int i = 0; i < n; ++i) {
    if (done[i] || !plans[i]->fast_compress) continue;
    const Variant v = {plans[i]->fast_S, plans[i]->fast_R, plans[i]->bf16 ? 1 : 0};
    std::vector<int> grp;
    for (int j = i; j < n && (int)grp.size() < maxb; ++j) {
      const asi_plan* q = plans[j];
      if (!done[j] && q->fast_compress && v == Variant{q->fast_S, q->fast_R, q->bf16 ? 1 : 0}) grp.push_back(j);
    }
    const int g = (int)grp.size();
    std::vector<SmPass1Args> pa(g);
    std::vector<SmReduceArgs> ra(g);
    std::vector<SmCoreArgs> ca(g);
    std::vector<int> mc(g);
    for (int k = 0; k < g; ++k) {
      const int j = grp[k];
      char* w = static_cast<char*>(ws[j]);
      build_fused_pass1(plans[j], acts[j], U_prev[j], w, &pa[k]);
      mc[k] = build_fused_reduce(plans[j], w, U_prev[j], &ra[k]);
      build_fused_core(plans[j], acts[j], U_new[j], cores[j], w, true, &ca[k]);
      done[j] = 1;
    }
    ASI_CUDA(launch_sm_pass1_batched(pa.data(), g, v.S, v.R, v.bf16 != 0, st));
    ASI_CUDA(launch_sm_reduce_batched(ra.data(), mc.data(), g, st));
    ASI_CUDA(launch_sm_core_batched(ca.data(), g, v.S, v.R, v.bf16 != 0, st));
  }
  for (int i = 0; i < n; ++i) {
    if (done[i]) continue;
    const asi_status_t s = asi_compress(plans[i], acts[i], U_prev[i], U_new[i], cores[i], ws[i], ws_bytes[i], stream);
    if (s != ASI_OK) return s;
  }
  return ASI_OK;
}

asi_status_t asi_wgrad_batched(const asi_plan_t* const* plans, const float* const* cores, const float* const* U,
                               const void* const* dY, float* const* dW, void* const* ws, const size_t* ws_bytes,
                               int32_t n, void* stream) {
  if (!plans || !cores || !U || !dY || !dW || !ws || !ws_bytes || n < 1 || n > 4096) return ASI_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    const asi_plan* pl = plans[i];
    if (!pl || !valid_ptr(cores[i]) || !valid_ptr(U[i]) || !valid_ptr(dY[i]) || !valid_ptr(dW[i]))
      return ASI_ERR_INVALID_ARG;
    const asi_status_t s = check_ws(ws[i], ws_bytes[i], pl->wgrad_ws);
    if (s != ASI_OK) return s;
    if (pl->fast_wgrad && pl->wgrad_bulk && (reinterpret_cast<uintptr_t>(dY[i]) & 15u)) return ASI_ERR_INVALID_ARG;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::vector<char> done(n, 0);
  const int maxb = sm_max_batch();
  for (int i = 0; i < n; ++i) {
    if (done[i] || !plans[i]->fast_wgrad) continue;
    const int R = plans[i]->fast_R, bf = plans[i]->bf16 ? 1 : 0;
    std::vector<SmWgradArgs> wa;
    for (int j = i; j < n && (int)wa.size() < maxb; ++j) {
      const asi_plan* q = plans[j];
      if (done[j] || !q->fast_wgrad || q->fast_R != R || (q->bf16 ? 1 : 0) != bf) continue;
      SmWgradArgs g;
      if (!build_fused_wgrad(q, cores[j], U[j], dY[j], dW[j], static_cast<char*>(ws[j]), &g))
        return ASI_ERR_INVALID_ARG;
      wa.push_back(g);
      done[j] = 1;
    }
    ASI_CUDA(launch_sm_wgrad_batched(wa.data(), (int)wa.size(), R, bf != 0, st));
  }
  for (int i = 0; i < n; ++i) {
    if (done[i]) continue;
    const asi_plan* pl = plans[i];
    const asi_status_t s = pl->d.kind == ASI_CONV2D
        ? asi_conv_wgrad(pl, cores[i], U[i], dY[i], dW[i], ws[i], ws_bytes[i], stream)
        : asi_linear_wgrad(pl, cores[i], U[i], dY[i], dW[i], ws[i], ws_bytes[i], stream);
    if (s != ASI_OK) return s;
  }
  return ASI_OK;
}

// ---------------------------------------------------------------------------------------------
// asi_compress with the workspace in the library image, for callers that may not allocate.
// g_static_ws names the array only in device code; host code must ask the runtime for its device
// address (once per device, with that device current) and hand that address to the kernels.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_ws[ASI_STATIC_WS_MAX_BYTES];

asi_status_t asi_compress_static_ws(const asi_plan_t* pl, const void* act, const float* U_prev,
                                    float* U_new, float* core, void* stream) {
  constexpr int kMaxDevices = 64;
  static void* addr_of_device[kMaxDevices] = {};
  static std::mutex setup_lock;
  if (!pl) return ASI_ERR_INVALID_ARG;
  if (pl->compress_ws > (size_t)ASI_STATIC_WS_MAX_BYTES) {
    snprintf(g_cuda_err, sizeof(g_cuda_err),
             "asi_compress_static_ws: the plan needs %zu bytes of scratch, the built-in array holds %u",
             pl->compress_ws, (unsigned)ASI_STATIC_WS_MAX_BYTES);
    return ASI_ERR_WORKSPACE;
  }
  int dev = -1;
  ASI_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ASI_ERR_UNSUPPORTED;
  void* ws = nullptr;
  {
    std::lock_guard<std::mutex> guard(setup_lock);
    if (!addr_of_device[dev]) {
      void* p = nullptr;
      ASI_CUDA(cudaGetSymbolAddress(&p, g_static_ws));
      addr_of_device[dev] = p;
    }
    ws = addr_of_device[dev];
  }
  // asi_compress clears the status word and the completion counters itself; everything else in the
  // array is written before it is read.
  return compress_impl(pl, act, U_prev, U_new, core, ws, (size_t)ASI_STATIC_WS_MAX_BYTES, stream, false);
}

asi_status_t asi_init_factors(const asi_plan_t* pl, const void* act, const float* omega, float* U_new,
                              float* core, void* ws, size_t ws_bytes, void* stream) {
  if (!pl || !valid_ptr(act) || !valid_ptr(omega) || !valid_ptr(U_new) || !valid_ptr(core))
    return ASI_ERR_INVALID_ARG;
  asi_status_t s = check_ws(ws, ws_bytes, pl->compress_ws);
  if (s != ASI_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if (pl->fast_compress && !pl->bf16 && (reinterpret_cast<uintptr_t>(act) & 15u)) return ASI_ERR_INVALID_ARG;
  ASI_CUDA(cudaMemsetAsync(w, 0, kStatusBytes, st));
  int64_t off = 0;
  for (int m = 0; m < pl->nd; ++m) {
    s = expand_mode(pl, m, act, omega + off, w, st);
    if (s != ASI_OK) return s;
    off += pl->mv[m].Q * pl->r[m];
  }
  return finish_compress(pl, act, U_new, core, w, nullptr, st);
}

static size_t omega_scratch_bytes(const asi_plan* pl) {
  int64_t mx = 0;
  for (int m = 0; m < pl->nd; ++m) mx = std::max<int64_t>(mx, pl->mv[m].Q * pl->r[m]);
  return align_up((size_t)mx * 4, 256);
}

size_t asi_init_seeded_ws_bytes(const asi_plan_t* pl) {
  return pl ? align_up(pl->compress_ws, 256) + omega_scratch_bytes(pl) : 0;
}

asi_status_t asi_init_factors_seeded(const asi_plan_t* pl, const void* act, uint64_t seed, float* U_new,
                                     float* core, void* ws, size_t ws_bytes, void* stream) {
  if (!pl || !valid_ptr(act) || !valid_ptr(U_new) || !valid_ptr(core)) return ASI_ERR_INVALID_ARG;
  asi_status_t s = check_ws(ws, ws_bytes, asi_init_seeded_ws_bytes(pl));
  if (s != ASI_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  float* omega = reinterpret_cast<float*>(w + align_up(pl->compress_ws, 256));
  if (pl->fast_compress && !pl->bf16 && (reinterpret_cast<uintptr_t>(act) & 15u)) return ASI_ERR_INVALID_ARG;
  ASI_CUDA(cudaMemsetAsync(w, 0, kStatusBytes, st));
  for (int m = 0; m < pl->nd; ++m) {               // one mode's Omega at a time, in the same scratch
    ASI_CUDA(launch_fill_gaussian(seed, (uint32_t)m, pl->mv[m].Q * pl->r[m], omega, st));
    s = expand_mode(pl, m, act, omega, w, st);
    if (s != ASI_OK) return s;
  }
  return finish_compress(pl, act, U_new, core, w, nullptr, st);
}

asi_status_t asi_gaussian_stream(uint64_t seed, uint32_t stream_id, int64_t n, float* out, void* stream) {
  if (n < 0 || (n > 0 && !valid_ptr(out))) return ASI_ERR_INVALID_ARG;
  ASI_CUDA(launch_fill_gaussian(seed, stream_id, n, out, static_cast<cudaStream_t>(stream)));
  return ASI_OK;
}

asi_status_t asi_philox_words(uint64_t seed, uint32_t stream_id, int64_t n_groups, uint32_t* out, void* stream) {
  if (n_groups < 0 || (n_groups > 0 && (!valid_ptr(out) || (reinterpret_cast<uintptr_t>(out) & 15u))))
    return ASI_ERR_INVALID_ARG;
  ASI_CUDA(launch_philox_words(seed, stream_id, n_groups, out, static_cast<cudaStream_t>(stream)));
  return ASI_OK;
}

asi_status_t asi_conv_wgrad(const asi_plan_t* pl, const float* core, const float* U, const void* dY,
                            float* dW, void* ws, size_t ws_bytes, void* stream) {
  if (!pl || !valid_ptr(core) || !valid_ptr(U) || !valid_ptr(dY) || !valid_ptr(dW))
    return ASI_ERR_INVALID_ARG;
  if (pl->d.kind != ASI_CONV2D) return ASI_ERR_INVALID_ARG;
  asi_status_t s = check_ws(ws, ws_bytes, pl->wgrad_ws);
  if (s != ASI_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if (pl->fast_wgrad) {
    SmWgradArgs g;
    if (!build_fused_wgrad(pl, core, U, dY, dW, w, &g)) return ASI_ERR_INVALID_ARG;
    ASI_CUDA(launch_sm_wgrad(g, pl->fast_R, pl->bf16, st));
    return ASI_OK;
  }
  float* Z1 = reinterpret_cast<float*>(w + pl->off_Z[0]);
  float* Z3a = reinterpret_cast<float*>(w + pl->off_Z[1]);
  float* Z3 = reinterpret_cast<float*>(w + pl->off_Z[2]);
  const int64_t B = pl->dims[0], H = pl->dims[2], W = pl->dims[3];
  const int r1 = pl->r[0], r2 = pl->r[1], r3 = pl->r[2], r4 = pl->r[3];
  const int64_t per_sample = (int64_t)pl->d.cout * pl->Ho * pl->Wo;

  ModeProdArgs a;
  // term 1: Z1 = dY x_1 U_1^T
  a.X = dY; a.B = U + pl->u_off[0]; a.Y = Z1;
  a.O = 1; a.a = B; a.I = per_sample; a.Q = per_sample;
  a.n_out = r1; a.ldb_k = r1; a.ldb_j = 1;
  a.so = (int64_t)r1 * per_sample; a.sj = per_sample; a.si = 1;
  ASI_CUDA(stream_modeprod(pl, a, pl->bf16, st));
  if (pl->conv_z3) {
    // terms 2-3 in one launch
    ASI_CUDA(launch_z3(core, U + pl->u_off[2], U + pl->u_off[3], Z3, r1 * r2, r3, r4, (int)H, (int)W, st));
  } else {
  // term 2: core x_3 U_3  -> [r1 r2, H, r4]
  a.X = core; a.B = U + pl->u_off[2]; a.Y = Z3a;
  a.O = (int64_t)r1 * r2; a.a = r3; a.I = r4; a.Q = a.O * a.I;
  a.n_out = (int)H; a.ldb_k = 1; a.ldb_j = r3;
  a.so = H * r4; a.sj = r4; a.si = 1;
  ASI_CUDA(launch_modeprod(a, false, st));
  // term 3: .. x_4 U_4 -> Z3 [r1 r2 H, W]
  a.X = Z3a; a.B = U + pl->u_off[3]; a.Y = Z3;
  a.O = (int64_t)r1 * r2 * H; a.a = r4; a.I = 1; a.Q = a.O;
  a.n_out = (int)W; a.ldb_k = 1; a.ldb_j = r4;
  a.so = W; a.sj = 1; a.si = 1;
  ASI_CUDA(launch_modeprod(a, false, st));
  }
  // terms 4 and 5
  ConvTailArgs t;
  t.Z1 = Z1; t.Z3 = Z3; t.U2 = U + pl->u_off[1]; t.dW = dW;
  t.r1 = r1; t.r2 = r2; t.C = (int)pl->dims[1]; t.Cout = pl->d.cout;
  t.H = (int)H; t.W = (int)W; t.Ho = (int)pl->Ho; t.Wo = (int)pl->Wo;
  t.kh = pl->d.kh; t.kw = pl->d.kw; t.sh = pl->d.stride_h; t.sw = pl->d.stride_w;
  t.ph = pl->d.pad_h; t.pw = pl->d.pad_w; t.groups = pl->d.groups;
  if (pl->conv_nsp > 1)
    ASI_CUDA(launch_conv_tail_split(t, reinterpret_cast<float*>(w + pl->off_Z4p), pl->conv_nsp, st));
  else
    ASI_CUDA(launch_conv_tail(t, st));
  return ASI_OK;
}

asi_status_t asi_linear_wgrad(const asi_plan_t* pl, const float* core, const float* U, const void* dY,
                              float* dW, void* ws, size_t ws_bytes, void* stream) {
  if (!pl || !valid_ptr(core) || !valid_ptr(U) || !valid_ptr(dY) || !valid_ptr(dW))
    return ASI_ERR_INVALID_ARG;
  if (pl->d.kind != ASI_LINEAR) return ASI_ERR_INVALID_ARG;
  asi_status_t s = check_ws(ws, ws_bytes, pl->wgrad_ws);
  if (s != ASI_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  const int nd = pl->nd, nlead = nd - 1;
  const int64_t Dout = pl->d.cout, Din = pl->dims[nd - 1];
  const int rl = pl->r[nd - 1];

  ModeProdArgs a;
  if (pl->lin_reorder) {
    // dY x_2 U_2^T on the tensor cores -> [B][Dout][r2], then x_1 U_1^T -> [r1][Dout][r2]
    const int64_t B = pl->dims[0], N = pl->dims[1];
    const int r1 = pl->r[0], r2 = pl->r[1];
    float* Y1 = reinterpret_cast<float*>(w + pl->off_Z[0]);
    float* Y2 = reinterpret_cast<float*>(w + pl->off_Z[1]);
    a.X = dY; a.B = U + pl->u_off[1]; a.Y = Y1;
    a.O = B; a.a = N; a.I = Dout; a.Q = B * Dout;
    a.n_out = r2; a.ldb_k = r2; a.ldb_j = 1;
    a.so = Dout * r2; a.sj = 1; a.si = r2;
    a.tc_scratch = w + pl->off_wtc; a.tc_scratch_bytes = pl->wtc_bytes;
    a.status = reinterpret_cast<int*>(w);
    ASI_CUDA(launch_modeprod(a, true, st));
    ModeProdArgs b;
    b.X = Y1; b.B = U + pl->u_off[0]; b.Y = Y2;
    b.O = 1; b.a = B; b.I = Dout * r2; b.Q = b.I;
    b.n_out = r1; b.ldb_k = r1; b.ldb_j = 1;
    b.so = (int64_t)r1 * b.I; b.sj = b.I; b.si = 1;
    b.status = reinterpret_cast<int*>(w);
    ASI_CUDA(stream_modeprod(pl, b, false, st));
    LinTailArgs t;
    t.Z = Y2; t.core = core; t.U = U + pl->u_off[2]; t.dW = dW;
    t.s1 = Dout * r2; t.s2 = 1; t.so = r2;
    t.L1 = r1; t.L2 = r2; t.Dout = (int)Dout; t.Din = (int)Din; t.r = rl; t.lead_fastest = 1;
    t.Z4p = reinterpret_cast<float*>(w + pl->off_Z[2]); t.nsplit = pl->lin_nsplit;
    ASI_CUDA(launch_lin_tail(t, st));
    return ASI_OK;
  }
  // Z = dY x_1 U_1^T (x_2 U_2^T): leading modes one by one
  int64_t cd[ASI_MAX_MODES];
  for (int m = 0; m < nlead; ++m) cd[m] = pl->dims[m];
  cd[nlead] = Dout;
  const void* src = dY;
  bool src_bf16 = pl->bf16;
  int64_t lead_r = 1;
  for (int m = 0; m < nlead; ++m) {
    a.X = src; a.B = U + pl->u_off[m];
    a.Y = reinterpret_cast<float*>(w + pl->off_Z[m]);
    a.O = 1; a.I = 1;
    for (int j = 0; j < m; ++j) a.O *= cd[j];
    for (int j = m + 1; j <= nlead; ++j) a.I *= cd[j];
    a.a = cd[m]; a.Q = a.O * a.I;
    a.n_out = pl->r[m]; a.ldb_k = pl->r[m]; a.ldb_j = 1;
    a.so = (int64_t)pl->r[m] * a.I; a.sj = a.I; a.si = 1;
    a.status = reinterpret_cast<int*>(w);
    ASI_CUDA(stream_modeprod(pl, a, src_bf16, st));
    cd[m] = pl->r[m];
    lead_r *= pl->r[m];
    src = a.Y;
    src_bf16 = false;
  }
  if (!(pl->d.flags & ASI_FLAG_GENERIC_ONLY)) {
    // Z4 = Z . core over the leading ranks and dW = Z4 U_last^T in one launch; Z is [r1 (r2)][Dout]
    LinTailArgs t;
    t.Z = static_cast<const float*>(src); t.core = core; t.U = U + pl->u_off[nd - 1]; t.dW = dW;
    t.L1 = pl->r[0]; t.L2 = (nlead > 1) ? pl->r[1] : 1;
    t.s1 = (int64_t)t.L2 * Dout; t.s2 = Dout; t.so = 1;
    t.Dout = (int)Dout; t.Din = (int)Din; t.r = rl; t.lead_fastest = 0;
    t.Z4p = reinterpret_cast<float*>(w + pl->off_Z[2]); t.nsplit = pl->lin_nsplit;
    ASI_CUDA(launch_lin_tail(t, st));
    return ASI_OK;
  }
  // Z4^T[k, o] = sum_{lead} Z[lead, o] core[lead, k]
  float* Z4t = reinterpret_cast<float*>(w + pl->off_Z[2]);
  a.X = src; a.B = core; a.Y = Z4t;
  a.O = 1; a.a = lead_r; a.I = Dout; a.Q = Dout;
  a.n_out = rl; a.ldb_k = rl; a.ldb_j = 1;
  a.so = 0; a.sj = Dout; a.si = 1;
  ASI_CUDA(launch_modeprod(a, false, st));
  // dW[o, d] = sum_k Z4^T[k, o] U_last[d, k]
  a.X = Z4t; a.B = U + pl->u_off[nd - 1]; a.Y = dW;
  a.O = 1; a.a = rl; a.I = Dout; a.Q = Dout;
  a.n_out = (int)Din; a.ldb_k = 1; a.ldb_j = rl;
  a.so = 0; a.sj = 1; a.si = Din;
  ASI_CUDA(launch_modeprod(a, false, st));
  return ASI_OK;
}

size_t asi_spectrum_ws_bytes(const asi_plan_t* pl) { return pl ? spectrum_ws_bytes(pl) : 0; }

asi_status_t asi_mode_spectrum(const asi_plan_t* pl, const void* act, double* eig, double* energy, void* ws,
                               size_t ws_bytes, void* stream) {
  if (!pl || !valid_ptr(act) || !eig || !energy) return ASI_ERR_INVALID_ARG;
  const asi_status_t s = check_ws(ws, ws_bytes, spectrum_ws_bytes(pl));
  if (s != ASI_OK) return s;
  ASI_CUDA(launch_mode_spectrum(pl, act, eig, energy, static_cast<char*>(ws), static_cast<cudaStream_t>(stream)));
  return ASI_OK;
}

asi_status_t asi_pick_ranks(const asi_plan_t* pl, const double* eig, const double* energy, double eps,
                            int32_t r_max, int32_t* ranks, void* stream) {
  if (!pl || !eig || !energy || !ranks || !(eps > 0.0) || !(eps <= 1.0) || r_max < 1) return ASI_ERR_INVALID_ARG;
  ASI_CUDA(launch_pick_ranks(pl, eig, energy, eps, r_max, ranks, static_cast<cudaStream_t>(stream)));
  return ASI_OK;
}

size_t asi_perplexity_ws_bytes(void) { return perplexity_ws_bytes(); }

asi_status_t asi_perplexity(const float* dW, const float* dW_approx, int64_t n, double* out, void* ws,
                            size_t ws_bytes, void* stream) {
  if (!dW || !dW_approx || !out || n < 1) return ASI_ERR_INVALID_ARG;
  const asi_status_t s = check_ws(ws, ws_bytes, perplexity_ws_bytes());
  if (s != ASI_OK) return s;
  ASI_CUDA(launch_perplexity(dW, dW_approx, n, out, static_cast<double*>(ws), static_cast<cudaStream_t>(stream)));
  return ASI_OK;
}

size_t asi_step_host_arena_bytes(const asi_plan_t* pl) {
  if (!pl) return 0;
  const size_t eb = elem_bytes(pl);
  size_t off = 0;
  off = align_up(off + (size_t)pl->N * eb, 256);
  off = align_up(off + (size_t)pl->dy_elems * eb, 256);
  off = align_up(off + (size_t)pl->u_elems * 4, 256) * 1;
  off = align_up(off + (size_t)pl->u_elems * 4, 256);
  off = align_up(off + (size_t)pl->core_elems * 4, 256);
  off = align_up(off + (size_t)pl->dw_elems * 4, 256);
  off += align_up(std::max(pl->compress_ws, pl->wgrad_ws), 256);
  return off;
}

asi_status_t asi_step_host(const asi_plan_t* pl, const void* act_host, const void* dY_host,
                           const float* U_prev_host, float* U_new_host, float* core_host,
                           float* dW_host, void* arena, size_t arena_bytes, void* stream) {
  if (!pl || !act_host || !dY_host || !U_prev_host || !U_new_host || !core_host || !dW_host)
    return ASI_ERR_INVALID_ARG;
  asi_status_t s = check_ws(arena, arena_bytes, asi_step_host_arena_bytes(pl));
  if (s != ASI_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t eb = elem_bytes(pl);
  char* base = static_cast<char*>(arena);
  size_t off = 0;
  char* d_act = base + off; off = align_up(off + (size_t)pl->N * eb, 256);
  char* d_dy = base + off; off = align_up(off + (size_t)pl->dy_elems * eb, 256);
  float* d_up = reinterpret_cast<float*>(base + off); off = align_up(off + (size_t)pl->u_elems * 4, 256);
  float* d_un = reinterpret_cast<float*>(base + off); off = align_up(off + (size_t)pl->u_elems * 4, 256);
  float* d_core = reinterpret_cast<float*>(base + off); off = align_up(off + (size_t)pl->core_elems * 4, 256);
  float* d_dw = reinterpret_cast<float*>(base + off); off = align_up(off + (size_t)pl->dw_elems * 4, 256);
  void* d_ws = base + off;
  const size_t ws_bytes = align_up(std::max(pl->compress_ws, pl->wgrad_ws), 256);
  ASI_CUDA(cudaMemcpyAsync(d_act, act_host, (size_t)pl->N * eb, cudaMemcpyHostToDevice, st));
  ASI_CUDA(cudaMemcpyAsync(d_up, U_prev_host, (size_t)pl->u_elems * 4, cudaMemcpyHostToDevice, st));
  s = asi_compress(pl, d_act, d_up, d_un, d_core, d_ws, ws_bytes, stream);
  if (s != ASI_OK) return s;
  ASI_CUDA(cudaMemcpyAsync(d_dy, dY_host, (size_t)pl->dy_elems * eb, cudaMemcpyHostToDevice, st));
  if (pl->d.kind == ASI_CONV2D)
    s = asi_conv_wgrad(pl, d_core, d_un, d_dy, d_dw, d_ws, ws_bytes, stream);
  else
    s = asi_linear_wgrad(pl, d_core, d_un, d_dy, d_dw, d_ws, ws_bytes, stream);
  if (s != ASI_OK) return s;
  ASI_CUDA(cudaMemcpyAsync(U_new_host, d_un, (size_t)pl->u_elems * 4, cudaMemcpyDeviceToHost, st));
  ASI_CUDA(cudaMemcpyAsync(core_host, d_core, (size_t)pl->core_elems * 4, cudaMemcpyDeviceToHost, st));
  ASI_CUDA(cudaMemcpyAsync(dW_host, d_dw, (size_t)pl->dw_elems * 4, cudaMemcpyDeviceToHost, st));
  return ASI_OK;
}

asi_status_t asi_step_host_status(const asi_plan_t* pl, const void* arena, void* stream,
                                  asi_status_t* device_status) {
  if (!pl || !arena || !device_status) return ASI_ERR_INVALID_ARG;
  const size_t eb = elem_bytes(pl);
  size_t off = 0;                                   // the same carve-up as asi_step_host
  off = align_up(off + (size_t)pl->N * eb, 256);
  off = align_up(off + (size_t)pl->dy_elems * eb, 256);
  off = align_up(off + (size_t)pl->u_elems * 4, 256);
  off = align_up(off + (size_t)pl->u_elems * 4, 256);
  off = align_up(off + (size_t)pl->core_elems * 4, 256);
  off = align_up(off + (size_t)pl->dw_elems * 4, 256);
  return asi_poll_status(pl, static_cast<const char*>(arena) + off, stream, device_status);
}

asi_status_t asi_profile_begin(int32_t kernel_id, void** events, int32_t n_pairs) {
  if (kernel_id < 1 || !events || n_pairs < 1) return ASI_ERR_INVALID_ARG;
  g_prof.ev = reinterpret_cast<cudaEvent_t*>(events);
  g_prof.n_pairs = n_pairs;
  g_prof.used = 0;
  g_prof.bytes = 0.0;
  g_prof.id = kernel_id;
  return ASI_OK;
}

int32_t asi_profile_end(double* alg_bytes) {
  const int used = g_prof.used;
  if (alg_bytes) *alg_bytes = g_prof.bytes;
  g_prof = ProfState{0, nullptr, 0, 0, 0.0};
  return used;
}

asi_status_t asi_poll_status(const asi_plan_t* pl, const void* ws, void* stream,
                             asi_status_t* device_status) {
  if (!pl || !ws || !device_status) return ASI_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int v = 0;
  ASI_CUDA(cudaMemcpyAsync(&v, ws, sizeof(int), cudaMemcpyDeviceToHost, st));
  ASI_CUDA(cudaStreamSynchronize(st));
  *device_status = static_cast<asi_status_t>(v);
  return ASI_OK;
}

}  // extern "C"
