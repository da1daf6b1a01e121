// Shared declarations of the CUDA library (host planning structs, K-order of the packed
// bf16 operand, small helpers).  Internal: the public contract is include/dc.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dc.h"

#define DC_CUDA_OK(expr)                        \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) return DC_ERR_CUDA; \
  } while (0)

static inline bool dc_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t dc_round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int dc_div_up(int a, int b) { return (a + b - 1) / b; }
static inline int dc_floor_div2(int a) { return (a >= 0) ? a / 2 : -((-a + 1) / 2); }

// Per-device host state.  SM counts and function attributes belong to a device, not to the process:
// both are kept per device ordinal (a process may drive several GPUs through the library).  The
// cached operations are idempotent, so two threads racing on a first use do no harm.
constexpr int kDcMaxDevices = 64;
static inline int dc_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kDcMaxDevices) return -1;
  return dev;
}
// SM count of the current device (148 when no device can be queried, e.g. host-only planning calls)
static inline int dc_sm_count() {
  static int cached[kDcMaxDevices];
  const int dev = dc_current_device();
  if (dev < 0) { (void)cudaGetLastError(); return 148; }
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}
// Raises a kernel's dynamic shared-memory limit once per device (`done` is the call site's own table).
template <typename K>
static inline cudaError_t dc_set_max_smem_once(K kernel, int bytes, unsigned char (&done)[kDcMaxDevices]) {
  const int dev = dc_current_device();
  if (dev >= 0 && done[dev]) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && dev >= 0) done[dev] = 1;
  return e;
}

static inline int dc_out_extent(int h, int k, int s, int p) {
  int a = h + 2 * p - k;
  return a < 0 ? 0 : a / s + 1;
}

// ----------------------------------------------------------------------------------------------
// K order of the packed bf16 weights (B operand) and of the activation planes (A operand).
//
// The reduction index of the implicit GEMM is cut into chunks of 8 input channels (16 bytes).
// A chunk entry is (column parity pc, channel chunk cc, tap row r, tap column s).  The input
// channels are processed in `ng` groups of `cg` chunks; inside a group the entries are ordered
// by (pc, cc, r, s) -- the order in which their shared-memory addresses increase -- and padded
// with one all-zero entry when their count is odd, because one tensor-core instruction consumes
// two entries (K = 16).  Stride 1 has a single parity; stride 2 splits the taps by the parity
// of the input column they read.
//
// "Fold" order (stride 1, k >= 3, few channels): the tap COLUMN s moves from K to N.  An entry is
// (chunk cc, tap row r) and the operand has k * co8 rows n = s * co8 + o (co8 = output channels
// rounded up to 8): one instruction then produces, for every tap column at once, the partial sums
// Z[m][s][o] = sum_{r,c} x[m + r * pitch][c] * W[o][c][r][s], and the epilogue adds the k column
// groups with a row shift, y[m][o] = sum_s Z[m + s][s][o].  This cuts the number of tensor-core
// instructions per output by k, which is what bounds small-channel convolutions.  With an odd
// number of entries the zero padding entry sits in front of the last one (positions e-1 and e), so
// that the activation side may pair the last entry with entry 0 read a second time -- a chunk that
// lies at a lower address, as the operand descriptor needs, and that always holds staged data.
//
// "Pair rows" order (stride 1, k >= 3, c_in <= 32, cheap enough): a GEMM row is a PAIR of
// neighbouring output pixels and the operand has 2 * co8 rows n = e * co8 + o, e = which pixel of
// the pair; the pair reads k+1 input columns, i.e. (k+1)/2 pairs of input pixels.  This costs
// (k+1)/2k more tensor-core work than plain order per output -- far less than it saves: half as
// many accumulator rows, and no reduction in the epilogue as fold order needs.  The GEMM is fed
// straight from TMA tiles: a shared-memory row is the
// 128-byte line of two neighbouring pixels (2 * c_in <= 64 channels, zero filled beyond), rows are
// 128-byte swizzled, and the K index of a row is simply its 16-byte chunks: chunk q holds
// elements 8q..8q+7 of (pixel 0 channels, pixel 1 channels).  An entry is (tap row r, pair shift t,
// chunk q); the weight of element (pixel px, channel c) of shift t for output pixel e of the pair
// is W[o][c][r][2t + px - e].  Nothing is repacked on the way in.
//
// Stride 2 (pair == 3) sits on the same lines with one output per GEMM row: output X reads the
// input columns 2X - pad + s, i.e. pixel px = (s + a) & 1 of pair shift t = (s + a) >> 1 with
// a = pad & 1 (the patch starts a pixels further left to keep pairs aligned); the operand has co8
// rows and the weight of element (px, c) of shift t is W[o][c][r][2t + px - a].
// ----------------------------------------------------------------------------------------------
struct KOrder {
  int k, stride, pad;
  int c_in, cch;      // input channels, chunks of 8 (rounded up)
  int cg, ng;         // chunks per group, groups
  int taps;           // k*k
  int pcs;            // 1 (stride 1) or 2 (stride 2)
  int ns[2];          // tap columns of each parity
  int s0[2];          // first tap column of each parity
  int e;              // entries per group = cg * taps
  int e_pad;          // e rounded up to even
  int n_pad;          // operand rows rounded up to 16 (output channels, or k * co8 in fold order)
  int fold;           // 1: fold order
  int pair;           // 2: pair rows (stride 1), 3: pair rows, stride 2
  int rows;           // 1: rows order (planes of 64 channels, passes of n_tile output channels)
  int n_tile, nnt;    // rows order: output channels per pass, passes (n_pad = nnt * n_tile)
  int co8;            // output channels rounded up to 8
};

static inline void dc_korder_init(KOrder *ko, const dc_geom *g) {
  ko->k = g->k; ko->stride = g->stride; ko->pad = g->pad;
  ko->c_in = g->c_in;
  ko->cch = dc_div_up(g->c_in, 8);
  ko->taps = g->k * g->k;
  ko->n_pad = (int)dc_round_up((size_t)g->c_out, 16);
  ko->co8 = (int)dc_round_up((size_t)g->c_out, 8);
  ko->fold = 0;
  ko->pair = 0;
  ko->rows = 0; ko->n_tile = 0; ko->nnt = 1;
  ko->pcs = (g->stride == 2) ? 2 : 1;
  if (g->groups == 1 && g->stride == 2 && g->k >= 3 && g->k <= 7 && ko->cch <= 4 && ko->co8 <= 128 &&
      g->c_in % 8 == 0 && g->c_out % 8 == 0) {
    const int a = g->pad & 1;
    const int nt = ((g->k - 1 + a) >> 1) + 1;
    const int n_pad = (int)dc_round_up((size_t)ko->co8, 16);
    if (g->k * nt * ko->cch <= 64 && (size_t)g->k * nt * 2 * ko->cch * n_pad * 16 <= 128 * 1024) {
      ko->pair = 3;
      ko->pcs = 1;
      ko->n_pad = n_pad;
      ko->ns[0] = nt; ko->ns[1] = 0; ko->s0[0] = 0; ko->s0[1] = 0;
      ko->cg = ko->cch; ko->ng = 1;
      ko->e = g->k * nt * 2 * ko->cch;
      ko->e_pad = ko->e;
      return;
    }
  }
  // pair rows (stride 1, 1x1 included) when their tensor-core cost stays small; beyond that fold
  // order (one instruction row per tap row) wins for narrow outputs
  // (1x1 layers with many output channels are bound by writing their output, which the general
  // kernel's staged bulk stores do better than this kernel's per-thread stores for wide outputs)
  if (g->groups == 1 && g->stride == 1 && g->k <= 7 && ko->cch <= 4 && ko->co8 <= (g->k == 1 ? 32 : 128) &&
      g->c_in % 8 == 0 && g->c_out % 8 == 0) {
    const int n_pad = (int)dc_round_up((size_t)(2 * ko->co8), 16);
    const int nt = (g->k + 1) / 2;
    if (g->k * nt * ko->cch <= 64 && (size_t)g->k * nt * 2 * ko->cch * n_pad * 16 <= 128 * 1024) {
      ko->pair = 2;
      ko->n_pad = n_pad;
      ko->ns[0] = nt; ko->ns[1] = 0; ko->s0[0] = 0; ko->s0[1] = 0;
      ko->cg = ko->cch; ko->ng = 1;
      ko->e = g->k * nt * 2 * ko->cch;
      ko->e_pad = ko->e;
      return;
    }
  }
  if (g->groups == 1 && g->stride == 1 && g->k >= 3 && g->k <= 7 && ko->cch <= 8 && ko->co8 <= 32 &&
      g->c_in % 8 == 0 && g->c_out % 8 == 0) {
    const int n_pad = (int)dc_round_up((size_t)(g->k * ko->co8), 16);
    if ((size_t)ko->cch * g->k * n_pad * 16 <= 64 * 1024) {
      ko->fold = 1;
      ko->n_pad = n_pad;
      ko->ns[0] = g->k; ko->ns[1] = 0; ko->s0[0] = 0; ko->s0[1] = 0;
      ko->cg = ko->cch; ko->ng = 1;
      ko->e = ko->cch * g->k;
      ko->e_pad = (ko->e + 1) & ~1;
      return;
    }
  }
  // rows order: stride 1, more channels than a pixel pair's line holds -- or, for k >= 3, more output channels
  // than the pair rows take (one half-filled plane then: 32 -> 192 3x3 at 28x28 measured 29 us here against
  // 37 us on the general kernel).  Chunk planes are
  // ordered (plane g of 64 channels, tap row r, tap column s, 16-channel step, half): the planes of
  // one (g, r) step are contiguous, which is the unit the kernel streams.
  if (g->groups == 1 && g->stride == 1 && g->k <= 7 &&
      (ko->cch >= 5 ? g->c_out >= 32
                    : ((g->k == 1 && ko->cch >= 2 && g->c_out >= 48) || (g->k >= 3 && ko->cch >= 2 && ko->co8 > 128))) &&
      g->c_in % 8 == 0 && g->c_out % 8 == 0) {
    const int n16 = (int)dc_round_up((size_t)g->c_out, 16);
    ko->rows = 1;
    // output channels per pass: at most 128, fewer for 5x5 and 7x7 kernels, whose weight stage of one
    // (plane, tap row) step (k * 8 chunk planes of n_tile rows) must fit the shared-memory ring twice
    // beside two activation stages and the epilogue's turn-around buffers
    const int n_tile_max = (g->k == 1 && g->c_in >= 512 && g->c_out > 256) ? 256 : (g->k <= 4 ? 128 : (g->k <= 5 ? 96 : 64));
    ko->nnt = dc_div_up(n16, n_tile_max);
    ko->n_tile = (int)dc_round_up((size_t)dc_div_up(n16, ko->nnt), 16);
    ko->n_pad = ko->nnt * ko->n_tile;
    ko->ns[0] = g->k; ko->ns[1] = 0; ko->s0[0] = 0; ko->s0[1] = 0;
    ko->cg = ko->cch; ko->ng = 1;
    const int steps = dc_div_up(g->c_in, 16);            // 16-channel steps over all planes
    ko->e = g->k * g->k * steps * 2;
    ko->e_pad = ko->e;
    return;
  }
  if (ko->pcs == 1) {
    ko->ns[0] = g->k; ko->ns[1] = 0; ko->s0[0] = 0; ko->s0[1] = 0;
  } else {
    for (int pc = 0; pc < 2; ++pc) {
      ko->s0[pc] = (g->pad + pc) & 1;
      ko->ns[pc] = (ko->s0[pc] >= g->k) ? 0 : (g->k - ko->s0[pc] + 1) / 2;
    }
  }
  // largest divisor of cch that is <= 8 and keeps one group's weights for <= 256 output
  // channels within 64 KB of shared memory
  int n_tile = ko->n_pad < 256 ? ko->n_pad : 256;
  int best = 1;
  for (int d = 1; d <= 8 && d <= ko->cch; ++d) {
    if (ko->cch % d) continue;
    if ((size_t)d * ko->taps * n_tile * 16 <= 96 * 1024) best = d;
  }
  ko->cg = best;
  ko->ng = ko->cch / best;
  ko->e = ko->cg * ko->taps;
  ko->e_pad = (ko->e + 1) & ~1;
}

// entry index within a group -> (pc, ccg, r, s); returns false for the zero padding entry
__host__ __device__ static inline bool dc_korder_decode(const KOrder &ko, int e, int *pc, int *ccg,
                                                        int *r, int *s) {
  if (ko.rows) {
    // plane g holds k * k * nsl(g) * 2 chunk planes, nsl = 4 except for a partial last plane
    if (e >= ko.e) return false;
    const int per_full = ko.k * ko.k * 8;
    const int gpl = e / per_full, rem = e - gpl * per_full;
    const int left = ko.c_in - 64 * gpl;
    const int nsl = left >= 64 ? 4 : (left + 15) / 16;
    const int half = rem & 1, q = rem >> 1;
    const int sl = q % nsl, tap = q / nsl;
    *r = tap / ko.k;
    *s = tap - *r * ko.k;
    *ccg = gpl * 8 + sl * 2 + half;
    *pc = 0;
    return true;
  }
  if (ko.pair >= 2) {
    // (tap row, pair shift, chunk of the pair row); *ccg returns the chunk, *s the shift
    if (e >= ko.e) return false;
    const int nq = 2 * ko.cch;
    *ccg = e % nq;
    const int u = e / nq;
    *s = u % ko.ns[0];
    *r = u / ko.ns[0];
    *pc = 0;
    return true;
  }
  if (ko.fold) {
    if (ko.e & 1) {
      if (e == ko.e - 1 || e > ko.e) return false;
      if (e == ko.e) e = ko.e - 1;
    } else if (e >= ko.e) {
      return false;
    }
    *pc = 0;
    *ccg = e / ko.k;
    *r = e - *ccg * ko.k;
    *s = -1;               // the tap column is part of the row index, not of the entry
    return true;
  }
  if (e >= ko.e) return false;
  if (ko.pcs == 1) {
    *pc = 0;
    *ccg = e / ko.taps;
    int t = e - *ccg * ko.taps;
    *r = t / ko.k;
    *s = t - *r * ko.k;
    return true;
  }
  int per0 = ko.k * ko.ns[0];
  int n0 = ko.cg * per0;
  int p = (e < n0) ? 0 : 1;
  int ee = (p == 0) ? e : e - n0;
  int per = ko.k * ko.ns[p];
  *pc = p;
  *ccg = ee / per;
  int rem = ee - *ccg * per;
  // tap rows in the order even rows, odd rows: the general kernel keeps the even and the odd patch rows
  // of a stride-2 layer apart, and the entries of a plane must come in the order of their addresses
  const int ri = rem / ko.ns[p], ne = (ko.k + 1) >> 1;
  *r = ri < ne ? 2 * ri : 2 * (ri - ne) + 1;
  *s = ko.s0[p] + 2 * (rem - ri * ko.ns[p]);
  return true;
}

// (channel chunk cc in [0,cch), tap r, s) -> position of that chunk in the packed weights,
// in units of chunk planes (n_pad * 8 elements each)
__host__ __device__ static inline int dc_korder_encode(const KOrder &ko, int cc, int r, int s) {
  if (ko.rows) {
    const int gpl = cc >> 3, left = ko.c_in - 64 * gpl;
    const int nsl = left >= 64 ? 4 : (left + 15) / 16;
    return gpl * ko.k * ko.k * 8 + ((r * ko.k + s) * nsl + ((cc & 7) >> 1)) * 2 + (cc & 1);
  }
  if (ko.pair == 2)            // the copy for the first pixel of the pair: dx = s, pixel s & 1 of shift s >> 1
    return (r * ko.ns[0] + (s >> 1)) * 2 * ko.cch + (s & 1) * ko.cch + cc;
  if (ko.pair == 3) {          // tap s sits at patch column s + a of the output's pair
    const int sa = s + (ko.pad & 1);
    return (r * ko.ns[0] + (sa >> 1)) * 2 * ko.cch + (sa & 1) * ko.cch + cc;
  }
  if (ko.fold) {
    const int e = cc * ko.k + r;
    return ((ko.e & 1) && e == ko.e - 1) ? e + 1 : e;
  }
  int grp = cc / ko.cg, ccg = cc - grp * ko.cg;
  int e;
  if (ko.pcs == 1) {
    e = ccg * ko.taps + r * ko.k + s;
  } else {
    int p = ((s - ko.pad) & 1);
    int per = ko.k * ko.ns[p];
    int base = (p == 0) ? 0 : ko.cg * ko.k * ko.ns[0];
    const int ri = (r & 1) ? ((ko.k + 1) >> 1) + (r >> 1) : (r >> 1);      // even tap rows first
    e = base + ccg * per + ri * ko.ns[p] + (s - ko.s0[p]) / 2;
  }
  return grp * ko.e_pad + e;
}

// Position (in 16-byte chunks of 8 channels) of row `row` of chunk plane `plane` in the packed weights.
// Planes are [n_pad rows][8 channels] one after the other, except in rows order with several output-
// channel passes: there a pass's n_tile rows of all planes are contiguous ([pass][plane][n_tile rows]),
// so that the planes of one (64-channel plane, tap row) step of one pass are one contiguous block.
__host__ __device__ static inline size_t dc_packed_chunk(const KOrder &ko, int plane, int row) {
  if (ko.rows && ko.nnt > 1) {
    const int pass = row / ko.n_tile;
    return ((size_t)pass * ko.e_pad + plane) * ko.n_tile + (row - pass * ko.n_tile);
  }
  return (size_t)plane * ko.n_pad + row;
}
// the inverse: chunk position -> (plane, row)
__host__ __device__ static inline void dc_packed_unchunk(const KOrder &ko, int idx8, int *plane, int *row) {
  if (ko.rows && ko.nnt > 1) {
    const int per_pass = ko.e_pad * ko.n_tile;
    const int pass = idx8 / per_pass, rem = idx8 - pass * per_pass;
    *plane = rem / ko.n_tile;
    *row = pass * ko.n_tile + (rem - *plane * ko.n_tile);
    return;
  }
  *plane = idx8 / ko.n_pad;
  *row = idx8 - *plane * ko.n_pad;
}

// row of output channel o (and tap column s) inside a chunk plane of the packed weights
__host__ __device__ static inline int dc_korder_row(const KOrder &ko, int s, int o) {
  return ko.fold ? s * ko.co8 + o : o;   // pair order: the first pixel's rows are 0..co8-1
}

__device__ __forceinline__ float dc_act_apply(float v, int act) {
  return act == DC_ACT_RELU6 ? fminf(fmaxf(v, 0.f), 6.f) : v;
}

// Programmatic dependent launch.  A kernel launched through dc_launch_pdl may be scheduled while the
// previous kernel of the stream is still running (its launch latency and start-up then overlap that
// kernel's end); it must call dc_pdl_enter() before it reads or writes global memory: that waits
// until the previous kernel has finished and its writes are visible, and lets the next kernel of
// the stream be scheduled in turn.  Launched in the ordinary way, the call returns at once.
__device__ __forceinline__ void dc_pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename... KArgs, typename... Args>
static inline cudaError_t dc_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                        Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Workspace header written by kernels with bounded waits.
struct DcWsHeader {
  unsigned int status;      // 0 or DC_ERR_TIMEOUT
  unsigned int where;       // which wait gave up
  unsigned int pad[62];
};

// internal launchers (defined in the .cu files)
dc_status dc_launch_conv_simt(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y,
                              dc_dtype dtype, cudaStream_t stream);
dc_status dc_launch_conv_tc(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                            const float *bias, dc_act act, const void *residual, void *y,
                            void *workspace, cudaStream_t stream);
bool dc_conv_tc_supported(int n, int h, int w, const dc_geom *g);
dc_status dc_launch_conv_pairrows(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                                  const float *bias, dc_act act, const void *residual, void *y,
                                  void *workspace, cudaStream_t stream);
bool dc_conv_pairrows_supported(int n, int h, int w, const dc_geom *g);
dc_status dc_launch_conv_rows(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y,
                              void *workspace, cudaStream_t stream);
bool dc_conv_rows_supported(int n, int h, int w, const dc_geom *g);
dc_status dc_launch_conv_fold(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y,
                              void *workspace, cudaStream_t stream);
bool dc_conv_fold_supported(int n, int h, int w, const dc_geom *g);
bool dc_conv_smallcin_supported(int n, int h, int w, const dc_geom *g);
dc_status dc_launch_conv_stem(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y,
                              void *workspace, cudaStream_t stream);
bool dc_conv_stem_supported(int n, int h, int w, const dc_geom *g);
dc_status dc_launch_conv_stem_s2(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                                 const float *bias, dc_act act, const void *residual, void *y,
                                 void *workspace, cudaStream_t stream);
bool dc_conv_stem_s2_supported(int n, int h, int w, const dc_geom *g);
bool dc_dwconv_stencil_supported(int n, int h, int w, int c, int k, int stride, int pad);
dc_status dc_launch_dwconv_stencil(const void *x, int n, int h, int w, int c, int k, int stride, int pad, const float *wp,
                                   const float *bias, dc_act act, void *y, cudaStream_t st);
dc_status dc_validate_geom(const dc_geom *g);
