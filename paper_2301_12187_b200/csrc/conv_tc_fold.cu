// Dense stride-1 convolution with few channels as an implicit GEMM whose tap COLUMNS are folded
// into the N dimension of the tensor-core instruction (see KOrder, "fold" order).
//
// Why: with 24..32 channels one tcgen05.mma of shape 128 x 32 x 16 does so little arithmetic that
// the kernel is bound by the number of instructions issued (measured: about 90 cycles per
// instruction from one issuing warp), not by HBM or the tensor pipe.  Folding the k tap columns
// into N turns k*k*cch/2 instructions per 128 output positions into k*cch/2 instructions of
// k-fold width:
//     Z[m][s][o] = sum_{r,c} x[m + r*pitch][c] * W[o][c][r][s]          (tensor core)
//     y[m][o]    = bias[o] + sum_s Z[m + s][s][o]                       (epilogue)
// The row shift m + s of the epilogue sum is a lane shift in tensor memory: __shfl_down inside a
// warp, a small shared-memory exchange across warp boundaries, and the last k-1 rows of each
// 128-row block are recomputed by the next block (blocks advance by 128-(k-1) positions).
//
// Staging is the chunk-plane scheme of conv_tc.cu: the haloed input patch of a tile is loaded
// once (16-byte cp.async, halo zero-filled) as planes of 8 channels at 16-byte pixel pitch, which
// is the no-swizzle K-major operand layout, so tap row r is the same plane read r*pitch pixels
// further on.  Weights arrive once per CTA by a 3-D TMA tile.  Output tiles go out with one bulk
// copy when they are contiguous in HBM.
//
// Roles (288 threads): warps 0-3 producers, warp 4 MMA issue (converged warp, elected lane) and
// tensor-memory owner, warps 5-8 epilogue.  Waits are bounded (tc::mbar_wait).
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kMaxStages = 8;
constexpr int kProducerThreads = 128;
constexpr int kThreads = 288;
constexpr int kMaxPieces = 8;   // 16-byte pieces of one patch row per producer thread

struct FoldParams {
  int n_img, h, w, ho, wo, c_in, c_out, co8;
  int k, pad, cch;
  int tw, th, nxt, wbox;       // tile size in outputs, x tiles per row, patch width (= GEMM row pitch)
  int n_pad;                   // N of the instruction: k column groups of co8 channels, padded
  int blk_rows;                // output positions per 128-row block = 128 - (k-1)
  int mb;                      // blocks per full tile
  int total_units;             // output row segments, ordered (img, xt, y)
  int plane_stride, a_stage_bytes, b_bytes;
  int stages, act, bulk_out, out_tile_bytes;
  int off_b, off_bias, off_out, off_xch, off_a, smem_bytes;
  int acc_cols, tmem_cols;
  int npairs, odd;
  uint32_t a_desc_lo[64];      // per instruction: (first chunk offset >> 4) | (distance >> 4) << 16
};

struct Tile {
  int img, xt, y0, th;
};

__device__ __forceinline__ Tile decode_tile(const FoldParams &p, int cur, int end) {
  Tile t;
  t.y0 = cur % p.ho;
  const int q = cur / p.ho;
  t.xt = q % p.nxt;
  t.img = q / p.nxt;
  int th = p.th;
  if (th > p.ho - t.y0) th = p.ho - t.y0;
  if (th > end - cur) th = end - cur;
  t.th = th;
  return t;
}

// Epilogue of one CTA (warps 5..8, 128 threads): for every tile, every 128-row block:
// read the k column groups of the accumulator, add them with their row shift, then bias, skip
// input, activation, bf16, and out (dense shared tile + one bulk copy, or 16-byte stores).
__device__ __forceinline__ void epilogue_role(const FoldParams &p, int cta_begin, int cta_end, uint32_t tmem_base,
                                              uint64_t *bar_accfull, uint64_t *bar_accempty,
                                              volatile uint32_t *abort_flag, DcWsHeader *ws, const float *bias_s,
                                              float *xch, uint8_t *smem_out, const __nv_bfloat16 *residual,
                                              __nv_bfloat16 *y) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = warp & 3;                        // tensor-memory lane quadrant this warp may read
  const bool elected = (threadIdx.x == 5 * 32);
  const int km1 = p.k - 1;
  // exchange buffer: [parity][quadrant][group s-1][lane < s][32 channels]
  const int xch_q = km1 * km1 * 32, xch_buf = 4 * xch_q;
  uint32_t it = 0, blk_count = 0;
  for (int cur = cta_begin; cur < cta_end; ++it) {
    const Tile t = decode_tile(p, cur, cta_end);
    cur += t.th;
    const int rows = (t.th - 1) * p.wbox + p.tw;
    const int nblk = (rows + p.blk_rows - 1) / p.blk_rows;
    const int x0 = t.xt * p.tw;
    const int tw_valid = (p.wo - x0 < p.tw) ? p.wo - x0 : p.tw;
    const uint32_t a = it & 1, aph = (it >> 1) & 1;
    uint8_t *obuf = smem_out + (size_t)a * p.out_tile_bytes;
    if (p.bulk_out && elected) bulk_wait_read1();   // the store that last used this buffer has read it
    // all 128 epilogue threads pass or leave together, so nobody is left alone at a named barrier
    if (!epi_all(mbar_wait(&bar_accfull[a], aph, abort_flag, ws, 0x40000u | a))) break;
    tc_fence_after();
    for (int b = 0; b < nblk; ++b, ++blk_count) {
      const int m = q * 32 + lane;
      const int pos = b * p.blk_rows + m;
      const int yy = pos / p.wbox, xx = pos - yy * p.wbox;
      const bool valid = (m < p.blk_rows) && (pos < rows) && (xx < tw_valid) && (yy < t.th);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * (uint32_t)p.acc_cols + (uint32_t)(b * p.n_pad);
      float *xw = xch + (blk_count & 1) * xch_buf;
      float acc[32];
      {
        uint32_t v[32];
        tmem_ld32(taddr, v);
        tmem_ld_wait();
#pragma unroll
        for (int o = 0; o < 32; ++o) acc[o] = __uint_as_float(v[o]);
      }
      for (int s = 1; s <= km1; ++s) {
        uint32_t v[32];
        tmem_ld32(taddr + (uint32_t)(s * p.co8), v);
        tmem_ld_wait();
        // rows handed to the previous warp: lanes 0..s-1 of this warp
        if (lane < s) {
          float *dst = xw + q * xch_q + ((s - 1) * km1 + lane) * 32;
#pragma unroll
          for (int o = 0; o < 32; o += 4)
            *reinterpret_cast<float4 *>(dst + o) = make_float4(__uint_as_float(v[o]), __uint_as_float(v[o + 1]),
                                                               __uint_as_float(v[o + 2]), __uint_as_float(v[o + 3]));
        }
        const bool take = lane + s < 32;
#pragma unroll
        for (int o = 0; o < 32; ++o) {
          const float tv = __shfl_down_sync(0xffffffffu, __uint_as_float(v[o]), s);
          if (take) acc[o] += tv;
        }
      }
      epi_barrier();                             // exchange rows are visible (buffers alternate per block)
      if (q < 3) {
        for (int s = 1; s <= km1; ++s) {
          if (lane + s >= 32) {
            const float *src = xw + (q + 1) * xch_q + ((s - 1) * km1 + (lane + s - 32)) * 32;
#pragma unroll
            for (int o = 0; o < 32; o += 4) {
              const float4 tv = *reinterpret_cast<const float4 *>(src + o);
              acc[o] += tv.x; acc[o + 1] += tv.y; acc[o + 2] += tv.z; acc[o + 3] += tv.w;
            }
          }
        }
      }
      if (valid) {
        const size_t pix = ((size_t)t.img * p.ho + (t.y0 + yy)) * p.wo + (x0 + xx);
        __nv_bfloat16 *gout = y + pix * p.c_out;
        const __nv_bfloat16 *gres = residual ? residual + pix * p.c_out : nullptr;
        uint8_t *sout = obuf + (size_t)(yy * p.tw + xx) * p.c_out * 2;
#pragma unroll
        for (int e8 = 0; e8 < 4; ++e8) {
          const int ch = e8 * 8;
          if (ch < p.c_out) {
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = acc[ch + i] + bias_s[ch + i];
            if (gres) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(gres + ch);
              const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 rf = __bfloat1622float2(rb[i]);
                f[2 * i] += rf.x; f[2 * i + 1] += rf.y;
              }
            }
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              ob[i] = __floats2bfloat162_rn(dc_act_apply(f[2 * i], p.act), dc_act_apply(f[2 * i + 1], p.act));
            if (p.bulk_out) *reinterpret_cast<uint4 *>(sout + ch * 2) = ov;
            else *reinterpret_cast<uint4 *>(gout + ch) = ov;
          }
        }
      }
    }
    tc_fence_before();
    mbar_arrive(&bar_accempty[a]);
    if (p.bulk_out) {
      fence_proxy_async();                       // the tile written above is read by the bulk copy engine
      epi_barrier();
      if (elected) {
        const size_t pix0 = ((size_t)t.img * p.ho + t.y0) * p.wo + x0;
        bulk_store(y + pix0 * p.c_out, smem_u32(obuf), (uint32_t)(t.th * p.tw * p.c_out * 2));
        bulk_commit();
      }
    }
  }
  if (p.bulk_out && elected) bulk_wait_all();
}

__device__ __forceinline__ void sync_consumers() { asm volatile("bar.sync 2, 160;" ::: "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
k_conv_tc_fold(const __grid_constant__ CUtensorMap map_b, const __grid_constant__ FoldParams p,
               const __nv_bfloat16 *__restrict__ x, const float *__restrict__ bias,
               const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_accfull[2], bar_accempty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ uint32_t abort_s;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *smem_b = smem + p.off_b;
  uint8_t *smem_a = smem + p.off_a;
  uint8_t *smem_out = smem + p.off_out;
  float *xch = reinterpret_cast<float *>(smem + p.off_xch);
  float *bias_s = reinterpret_cast<float *>(smem + p.off_bias);
  uint8_t *smem_zero = smem_a + (size_t)p.stages * p.a_stage_bytes;   // always-zero plane + slack

  const int warp = threadIdx.x >> 5;
  volatile uint32_t *abort_flag = &abort_s;

  // ---- set-up.  Producers only need the barriers, so they are released first; the consumers
  // (MMA + epilogue warps) finish their own preparation behind a second barrier.
  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < p.stages; ++s) { mbar_init(&bar_full[s], kProducerThreads); mbar_init(&bar_empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bar_accfull[a], 1); mbar_init(&bar_accempty[a], 128); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tensormap(&map_b);
  }
  __syncthreads();

  const int cta_begin = (int)((long long)p.total_units * blockIdx.x / gridDim.x);
  const int cta_end = (int)((long long)p.total_units * (blockIdx.x + 1) / gridDim.x);

  if (warp < 4) {
    // ================================================================== producers
    const int ptid = threadIdx.x;
    const int row_pieces = p.wbox * p.cch;      // 16-byte pieces per patch row; piece q = (col, chunk)
    const int C2 = p.c_in * 2;
    const int npieces = (ptid < row_pieces) ? (row_pieces - ptid + kProducerThreads - 1) / kProducerThreads : 0;
    int col_of[kMaxPieces];
    uint32_t dst_off[kMaxPieces];
#pragma unroll
    for (int i = 0; i < kMaxPieces; ++i) {
      if (i >= npieces) break;
      const int q = ptid + i * kProducerThreads;
      const int cc = q % p.cch;
      col_of[i] = q / p.cch;
      dst_off[i] = (uint32_t)(cc * p.plane_stride + col_of[i] * 16);
    }
    const uint32_t a_base0 = smem_u32(smem_a);
    const long long row_stride = (long long)p.w * C2;
    const uint32_t drow_stride = (uint32_t)p.wbox * 16u;
    uint32_t it = 0;
    bool ok = true;
    for (int cur = cta_begin; cur < cta_end && ok; ++it) {
      const Tile t = decode_tile(p, cur, cta_end);
      cur += t.th;
      const int gx0 = t.xt * p.tw - p.pad;
      const int gy0 = t.y0 - p.pad;
      const int rows = t.th + p.k - 1;
      const int r_lo = gy0 < 0 ? -gy0 : 0;                       // patch rows [r_lo, r_hi) lie inside the image
      const int r_hi = (p.h - gy0 < rows) ? p.h - gy0 : rows;
      // pieces of a pixel row are contiguous in memory: piece q sits 16*q bytes after the row start
      const char *tile_base = reinterpret_cast<const char *>(x) + (size_t)t.img * p.h * row_stride +
                              ((long long)gy0 * p.w + gx0) * C2 + (long long)ptid * 16;
      const int s = it % p.stages;
      const uint32_t ph = (it / p.stages) & 1;
      if (!mbar_wait(&bar_empty[s], ph ^ 1, abort_flag, ws, 0x10000u | s)) { ok = false; break; }
      if (ptid == 0 && it == 0) {
        // the weights ride on the first stage's barrier as transaction bytes and stay resident
        mbar_expect_tx(&bar_full[0], (uint32_t)p.b_bytes);
        tma_load_3d(smem_b, &map_b, &bar_full[0], 0, 0, 0);
      }
      const uint32_t stage = a_base0 + (uint32_t)s * p.a_stage_bytes;
#pragma unroll
      for (int i = 0; i < kMaxPieces; ++i) {
        if (i >= npieces) break;
        const int gx = gx0 + col_of[i];
        const bool cv = (gx >= 0) && (gx < p.w);
        const char *src = tile_base + (long long)i * (kProducerThreads * 16);
        uint32_t dst = stage + dst_off[i];
        for (int r = 0; r < rows; ++r) {
          const bool v = cv && (r >= r_lo) && (r < r_hi);
          cp_async16(dst, v ? (const void *)src : (const void *)x, v ? 16u : 0u);
          src += row_stride;
          dst += drow_stride;
        }
      }
      cp_async_arrive(&bar_full[s]);             // arrives by itself when this thread's copies have landed
    }
    cp_async_wait_all();                         // nothing of this thread is in flight when the CTA leaves
  } else {
    // ---- consumer preparation
    if (warp == 4) {
      tmem_alloc(&tmem_base_s, (uint32_t)p.tmem_cols);
      tmem_relinquish();
    } else {
      const int t = threadIdx.x - 5 * 32;
      for (int i = t; i < 32; i += 128) bias_s[i] = (bias && i < p.c_out) ? bias[i] : 0.f;
      uint4 *z = reinterpret_cast<uint4 *>(smem_zero);
      for (int i = t; i < (p.mb * 2048 + 1024) / 16; i += 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
      fence_proxy_async();
    }
    tc_fence_before();
    sync_consumers();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    if (warp == 4) {
      // ================================================================== MMA issue
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pad >> 3) << 17) | (8u << 24);
      const uint32_t desc_hi = (128u >> 4) | (1u << 14);
      const uint32_t zero_addr = smem_u32(smem_zero);
      const uint32_t b_base = smem_u32(smem_b);
      const uint32_t b_lo0 = ((b_base >> 4) & 0x3FFFu) | ((uint32_t)p.n_pad << 16);
      const uint32_t b_step = 2u * (uint32_t)p.n_pad;
      const uint32_t last = (uint32_t)(p.npairs - 1);
      const uint32_t first_off = (p.a_desc_lo[last] & 0x3FFFu) << 4;
      uint32_t it = 0;
      for (int cur = cta_begin; cur < cta_end; ++it) {
        const Tile t = decode_tile(p, cur, cta_end);
        cur += t.th;
        const int rows = (t.th - 1) * p.wbox + p.tw;
        const int nblk = (rows + p.blk_rows - 1) / p.blk_rows;
        const uint32_t a = it & 1, aph = (it >> 1) & 1;
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!warp_wait(&bar_accempty[a], aph ^ 1, abort_flag, ws, 0x20000u | a)) break;
        if (!warp_wait(&bar_full[s], ph, abort_flag, ws, 0x30000u | s)) break;
        tc_fence_after();
        const uint32_t a_base = smem_u32(smem_a + (size_t)s * p.a_stage_bytes);
        // last pair of an odd entry count: its second chunk is the zero plane
        const uint32_t pad_lo = (first_off >> 4) | (((zero_addr - a_base - first_off) >> 4) << 16);
        for (int b = 0; b < nblk; ++b) {
          const uint32_t d = tmem_base + a * (uint32_t)p.acc_cols + (uint32_t)(b * p.n_pad);
          const uint32_t a_add = (a_base >> 4) + (uint32_t)(b * p.blk_rows);
#pragma unroll 2
          for (int j = 0; j < p.npairs; ++j) {
            uint32_t lo = p.a_desc_lo[j];
            if (p.odd && (uint32_t)j == last) lo = pad_lo;
            const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(lo + a_add);
            const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo0 + (uint32_t)j * b_step);
            if (elect_one()) umma_bf16(d, ad, bd, idesc, j != 0 ? 1u : 0u);
          }
        }
        if (elect_one()) {
          umma_commit(&bar_empty[s]);            // the stage may be refilled once these MMAs finish
          umma_commit(&bar_accfull[a]);          // and the accumulators are complete
        }
      }
    } else {
      epilogue_role(p, cta_begin, cta_end, tmem_base, bar_accfull, bar_accempty, abort_flag, ws, bias_s, xch,
                    smem_out, residual, y);
    }
    // ---- consumer teardown
    if (*abort_flag) {
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    sync_consumers();
    if (warp == 4) {
      tc_fence_after();
      tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
  }
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

constexpr int kSmemBudget = 200 * 1024;

// plane stride in 16-byte units, chosen so that the chunks of one pixel (written by neighbouring
// producer threads) fall into different bank groups
int padded_plane_units(int units, int cch) {
  int want = (cch == 3 || cch == 5 || cch == 7) ? cch : (cch >= 8 ? 1 : (8 / cch));
  while ((units & 7) != (want & 7)) ++units;
  return units;
}

bool fold_plan(int n, int h, int w, const dc_geom *g, int n_sm, FoldParams *p) {
  KOrder ko;
  dc_korder_init(&ko, g);
  if (!ko.fold) return false;
  const int ho = dc_out_extent(h, g->k, 1, g->pad), wo = dc_out_extent(w, g->k, 1, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  if ((long long)n * h * w * g->c_in >= (1ll << 40)) return false;
  p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
  p->c_in = g->c_in; p->c_out = g->c_out; p->co8 = ko.co8;
  p->k = g->k; p->pad = g->pad; p->cch = ko.cch;
  p->n_pad = ko.n_pad;
  p->blk_rows = 128 - (g->k - 1);
  p->npairs = ko.e_pad / 2;
  p->odd = ko.e & 1;
  if (p->npairs > 64) return false;
  int mb_max = 256 / p->n_pad;
  if (mb_max > 4) mb_max = 4;
  if (mb_max < 1) return false;
  const int nxt = dc_div_up(wo, 64);
  p->tw = dc_div_up(wo, nxt);
  p->nxt = dc_div_up(wo, p->tw);
  p->wbox = p->tw + g->k - 1;
  if (p->wbox * p->cch > kMaxPieces * kProducerThreads) return false;
  // rows per tile: bounded by the accumulator blocks, the image, shared memory, and a target of
  // about six tiles per CTA so that load, MMA and epilogue overlap
  const long long total_rows = (long long)n * ho * p->nxt;
  if (total_rows >= (1ll << 31)) return false;
  int th_target = (int)(total_rows / ((long long)n_sm * 6));
  if (th_target < 1) th_target = 1;
  int th = (mb_max * p->blk_rows - p->tw) / p->wbox + 1;
  if (th < 1) return false;
  if (th > ho) th = ho;
  if (th > th_target) th = th_target;
  while (th > 1 && (long long)p->cch * ((th + g->k - 1) * p->wbox + 8) * 16 > 40 * 1024) --th;
  p->th = th;
  const int rbox = th + g->k - 1;
  p->mb = dc_div_up((th - 1) * p->wbox + p->tw, p->blk_rows);
  if (p->mb > mb_max) return false;
  p->plane_stride = padded_plane_units(rbox * p->wbox + 1, p->cch) * 16;
  p->a_stage_bytes = (int)dc_round_up((size_t)p->cch * p->plane_stride, 128);
  p->b_bytes = ko.e_pad * p->n_pad * 16;
  p->acc_cols = p->mb * p->n_pad;
  int cols = 32;
  while (cols < 2 * p->acc_cols) cols *= 2;
  if (cols > 512) return false;
  p->tmem_cols = cols;
  p->total_units = (int)total_rows;
  p->out_tile_bytes = (int)dc_round_up((size_t)th * p->tw * g->c_out * 2, 128);
  p->bulk_out = (p->tw == wo && p->out_tile_bytes <= 24 * 1024) ? 1 : 0;
  if (!p->bulk_out) p->out_tile_bytes = 0;
  const int km1 = g->k - 1;
  const int xch_bytes = 2 * 4 * km1 * km1 * 32 * 4;
  const int slack = p->mb * 2048 + 1024;
  p->off_b = 0;
  p->off_bias = (int)dc_round_up((size_t)p->b_bytes, 128);
  p->off_out = p->off_bias + 128;
  p->off_xch = p->off_out + 2 * p->out_tile_bytes;
  p->off_a = (int)dc_round_up((size_t)p->off_xch + xch_bytes, 128);
  long long per_cta = total_rows / th / n_sm + 2;
  int stages = kMaxStages;
  if (stages > per_cta) stages = (int)per_cta;
  while (stages >= 2 && 1024ll + p->off_a + (long long)stages * p->a_stage_bytes + slack > kSmemBudget) --stages;
  if (stages < 2) return false;
  p->stages = stages;
  p->smem_bytes = 1024 + p->off_a + stages * p->a_stage_bytes + slack;
  // chunk-pair table: entry e = (chunk cc, tap row r) -> byte offset of its 16-byte column in a stage
  for (int j = 0; j < p->npairs; ++j) {
    uint32_t off[2] = {0u, 16u};
    for (int q = 0; q < 2; ++q) {
      int pc, ccg, r, s;
      if (dc_korder_decode(ko, 2 * j + q, &pc, &ccg, &r, &s))
        off[q] = (uint32_t)(ccg * p->plane_stride + r * p->wbox * 16);
      else if (q == 1)
        off[1] = off[0] + 16;
    }
    p->a_desc_lo[j] = (off[0] >> 4) | (((off[1] - off[0]) >> 4) << 16);
  }
  return true;
}

}  // namespace

bool dc_conv_fold_supported(int n, int h, int w, const dc_geom *g) {
  FoldParams p;
  return fold_plan(n, h, w, g, 148, &p);
}

dc_status dc_launch_conv_fold(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                              cudaStream_t stream) {
  FoldParams p;
  const int n_sm = sm_count();
  if (!fold_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return DC_ERR_CUDA;
  CUtensorMap map_b;
  {
    const int e_pad = p.npairs * 2;
    cuuint64_t gdim[3] = {8, (cuuint64_t)p.n_pad, (cuuint64_t)e_pad};
    cuuint64_t gstr[2] = {16, (cuuint64_t)p.n_pad * 16};
    cuuint32_t box[3] = {8, (cuuint32_t)p.n_pad, (cuuint32_t)e_pad};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(w_packed), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  static bool attr_set = false;
  if (!attr_set) {
    DC_CUDA_OK(cudaFuncSetAttribute(k_conv_tc_fold, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    attr_set = true;
  }
  int grid = p.total_units < n_sm ? p.total_units : n_sm;
  k_conv_tc_fold<<<grid, kThreads, p.smem_bytes, stream>>>(map_b, p, (const __nv_bfloat16 *)x, bias,
                                                          (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                                          (DcWsHeader *)workspace);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
