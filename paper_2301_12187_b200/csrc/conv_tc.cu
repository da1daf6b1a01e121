// Dense convolution forward as an implicit GEMM on the 5th-generation tensor cores (sm_100a):
// tcgen05.mma with the accumulator in tensor memory, operands staged in shared memory by TMA.
//
// GEMM view.  M = output pixels of a tile, N = output channels, K = (tap, input channel).
// The activation tile is loaded ONCE per (tile, channel group) as a haloed patch and kept in
// shared memory as "chunk planes": plane (cc) holds, for every pixel of the patch, the 8
// channels [8cc, 8cc+8) as one 16-byte unit.  With 16-byte pixel pitch the no-swizzle K-major
// operand layout of tcgen05 (8 rows x 16 bytes core matrices, rows 16 bytes apart) is exactly a
// run of consecutive pixels, so the A operand of tap (r, s) is the same plane read from a start
// address shifted by (r * patch_width + s) pixels: no im2col copy and no reload per tap.  Rows
// of the GEMM enumerate the patch row-major INCLUDING its halo columns (pitch P), so a shifted
// view stays a constant offset; rows that fall on halo columns are computed and dropped.
// Stride 2 splits the patch by input-column parity (two sets of planes at half resolution).
//
// One tensor-core instruction takes K = 16 = two 16-byte chunks, addressed as "start" and
// "start + LBO": any two chunk entries whose addresses increase can be paired, which is how
// channel counts that are not multiples of 16 (24 = 3 chunks) avoid padding.
//
// Roles per CTA (192 threads): warp 0 lane 0 issues TMA loads into a ring of stages; warp 1
// lane 0 issues the MMAs and owns the tensor-memory allocation; warps 2..5 read accumulators
// back (tcgen05.ld), add bias / skip input, apply the activation and store bf16 NHWC.
// Accumulators are double buffered so the epilogue of tile i overlaps the MMAs of tile i+1.
// Every wait is bounded: when one runs out the CTA latches DC_ERR_TIMEOUT and leaves.
#include <cuda.h>

#include "common.cuh"

namespace {

constexpr int kMaxStages = 8;
constexpr int kThreads = 192;
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s per wait

struct TcParams {
  int n_img, h, w, ho, wo, c_out;
  int stride;
  int tw, th, nxt;            // tile width / height in outputs, x tiles per row
  int P, mb;                  // GEMM-row pitch per output row, 128-row blocks per tile
  int n_tile, nnt;            // output channels per pass, passes
  int units_per_nt, total_units;
  int cg, ng, e_pad, cch, pcs;
  int wbox, rbox;             // TMA box: patch columns, rows
  int plane_bytes, region_bytes, a_stage_bytes, b_stage_bytes;
  int stages, b_resident;
  int act;
  int cx0, cy0;               // patch origin: x = xt*tw + cx0, y = y0*stride + cy0
  int acc_cols, tmem_cols;
  int smem_bytes;
  KOrder ko;
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try(uint64_t *bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done;
}

// Bounded wait.  Returns false when the wait ran out (or another role already gave up).
__device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                            DcWsHeader *ws, uint32_t site) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 32; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > kWaitLimitNs) {
      *abort_flag = 1;
      atomicExch(&ws->status, (unsigned int)DC_ERR_TIMEOUT);
      ws->where = site;
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          DcWsHeader *ws, uint32_t site) {
  for (int i = 0; i < 16; ++i)
    if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, ws, site);
}

__device__ __forceinline__ void tma_load_5d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
      "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], M = 128, N from idesc, K = 16, bf16 in / fp32 out
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on an mbarrier once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 lanes x 16 consecutive fp32 columns: thread i of the warp receives lane (base lane + i)
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t *v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(addr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared-memory operand descriptor, K-major, no swizzle: 14-bit start>>4, LBO>>4 at bit 16,
// SBO>>4 at bit 32, descriptor version 1 at bit 46
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes) {
  const uint32_t lo = ((addr >> 4) & 0x3FFFu) | ((lbo_bytes >> 4) << 16);
  const uint32_t hi = (128u >> 4) | (1u << 14);
  return ((uint64_t)hi << 32) | lo;
}

// ------------------------------------------------------------------------------------------ tiles
struct Tile {
  int nt, img, xt, y0, th;
};

__device__ __forceinline__ Tile decode_tile(const TcParams &p, int cur, int end) {
  Tile t;
  t.nt = cur / p.units_per_nt;
  int rem = cur - t.nt * p.units_per_nt;
  t.y0 = rem % p.ho;
  int q = rem / p.ho;
  t.xt = q % p.nxt;
  t.img = q / p.nxt;
  int th = p.th;
  if (th > p.ho - t.y0) th = p.ho - t.y0;
  if (th > end - cur) th = end - cur;
  t.th = th;
  return t;
}

// ------------------------------------------------------------------------------------------ kernel
__global__ void __launch_bounds__(kThreads, 1)
k_conv_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
          const __grid_constant__ TcParams p, const float *__restrict__ bias,
          const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_accfull[2], bar_accempty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ uint32_t abort_s;
  __shared__ uint32_t a_off[128];   // per instruction j: byte offset of its first chunk in the stage
  __shared__ uint32_t a_lbo[128];   // per instruction j: byte distance to its second chunk

  // dynamic shared memory: [B stages][A stages][slack], 1024-byte aligned base
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int nb = p.b_resident ? 1 : p.stages;
  uint8_t *smem_b = smem;
  uint8_t *smem_a = smem + (size_t)nb * p.b_stage_bytes;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t *abort_flag = &abort_s;

  // ---- set-up
  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < p.stages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bar_accfull[a], 1); mbar_init(&bar_accempty[a], 128); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  // chunk-pair table: entry e -> byte offset of its 16-byte column in an A stage
  for (int j = threadIdx.x; j < p.e_pad / 2; j += kThreads) {
    uint32_t off[2];
    for (int q = 0; q < 2; ++q) {
      int e = 2 * j + q, pc, ccg, r, s;
      if (dc_korder_decode(p.ko, e, &pc, &ccg, &r, &s)) {
        int sx = (p.stride == 1) ? s : ((s - p.ko.pad) >> 1) - ((-p.ko.pad) >> 1);
        off[q] = (uint32_t)(pc * p.region_bytes + ccg * p.plane_bytes + (r * p.wbox + sx) * 16);
      } else {
        off[q] = off[0] + 16;  // zero-weight padding entry: any finite data will do
      }
    }
    a_off[j] = off[0];
    a_lbo[j] = off[1] - off[0];
  }
  // the bytes between the end of the planes and the end of each region are never written by
  // TMA but can be read through the padding entry: make them zero once
  {
    const int used = p.cg * p.plane_bytes, padb = p.region_bytes - used;
    const int nreg = p.stages * p.pcs;
    for (int i = threadIdx.x; i < nreg * (padb / 4); i += kThreads) {
      int reg = i / (padb / 4), wd = i - reg * (padb / 4);
      int st = reg / p.pcs, pc = reg - st * p.pcs;
      *reinterpret_cast<uint32_t *>(smem_a + (size_t)st * p.a_stage_bytes + pc * p.region_bytes + used + wd * 4) = 0u;
    }
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_s, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  const int cta_begin = (int)((long long)p.total_units * blockIdx.x / gridDim.x);
  const int cta_end = (int)((long long)p.total_units * (blockIdx.x + 1) / gridDim.x);

  if (warp == 0) {
    // ================================================================== producer (TMA)
    if (lane == 0) {
      const uint32_t a_bytes = (uint32_t)(p.pcs * p.cg * p.plane_bytes);
      uint32_t it = 0;
      bool b_loaded = false;
      for (int cur = cta_begin; cur < cta_end;) {
        const Tile t = decode_tile(p, cur, cta_end);
        cur += t.th;
        const int cx = t.xt * p.tw + p.cx0, cy = t.y0 * p.stride + p.cy0;
        for (int grp = 0; grp < p.ng; ++grp, ++it) {
          const int s = it % p.stages;
          const uint32_t ph = (it / p.stages) & 1;
          if (!mbar_wait(&bar_empty[s], ph ^ 1, abort_flag, ws, 0x10000u | s)) goto producer_done;
          const bool load_b = !p.b_resident || !b_loaded;
          mbar_expect_tx(&bar_full[s], a_bytes + (load_b ? (uint32_t)p.b_stage_bytes : 0u));
          uint8_t *dst = smem_a + (size_t)s * p.a_stage_bytes;
          for (int pc = 0; pc < p.pcs; ++pc)
            tma_load_5d(dst + pc * p.region_bytes, &map_a, &bar_full[s], 0, cx, cy, t.img, pc * p.cch + grp * p.cg);
          if (load_b) {
            tma_load_3d(smem_b + (size_t)(p.b_resident ? 0 : s) * p.b_stage_bytes, &map_b, &bar_full[s], 0,
                        t.nt * p.n_tile, grp * p.e_pad);
            b_loaded = true;
          }
        }
      }
    }
  producer_done:;
  } else if (warp == 1) {
    // ================================================================== MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_tile >> 3) << 17) | (8u << 24);
      const uint32_t b_lbo = (uint32_t)p.n_tile * 16u;
      const int npairs = p.e_pad / 2;
      uint32_t it = 0, tile_i = 0;
      for (int cur = cta_begin; cur < cta_end; ++tile_i) {
        const Tile t = decode_tile(p, cur, cta_end);
        cur += t.th;
        const int rows = (t.th - 1) * p.P + p.tw;
        const int nblk = (rows + 127) >> 7;
        const uint32_t a = tile_i & 1, aph = (tile_i >> 1) & 1;
        if (!mbar_wait(&bar_accempty[a], aph ^ 1, abort_flag, ws, 0x20000u | a)) goto mma_done;
        tc_fence_after();
        const uint32_t d0 = tmem_base + a * (uint32_t)p.acc_cols;
        for (int grp = 0; grp < p.ng; ++grp, ++it) {
          const int s = it % p.stages;
          const uint32_t ph = (it / p.stages) & 1;
          if (!mbar_wait(&bar_full[s], ph, abort_flag, ws, 0x30000u | s)) goto mma_done;
          tc_fence_after();
          const uint32_t a_base = smem_u32(smem_a + (size_t)s * p.a_stage_bytes);
          const uint32_t b_base = smem_u32(smem_b + (size_t)(p.b_resident ? 0 : s) * p.b_stage_bytes);
          for (int b = 0; b < nblk; ++b) {
            const uint32_t d = d0 + (uint32_t)(b * p.n_tile);
            for (int j = 0; j < npairs; ++j) {
              const uint64_t ad = make_desc(a_base + a_off[j] + (uint32_t)b * 2048u, a_lbo[j]);
              const uint64_t bd = make_desc(b_base + (uint32_t)(2 * j) * b_lbo, b_lbo);
              umma_bf16(d, ad, bd, idesc, (grp | j) != 0 ? 1u : 0u);
            }
          }
          umma_commit(&bar_empty[s]);            // stage s may be refilled once these MMAs finish
        }
        umma_commit(&bar_accfull[a]);            // accumulator a is complete
      }
    }
  mma_done:;
  } else {
    // ================================================================== epilogue (4 warps)
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    uint32_t tile_i = 0;
    for (int cur = cta_begin; cur < cta_end; ++tile_i) {
      const Tile t = decode_tile(p, cur, cta_end);
      cur += t.th;
      const int rows = (t.th - 1) * p.P + p.tw;
      const int nblk = (rows + 127) >> 7;
      const int x0 = t.xt * p.tw;
      const int tw_valid = (p.wo - x0 < p.tw) ? p.wo - x0 : p.tw;
      const uint32_t a = tile_i & 1, aph = (tile_i >> 1) & 1;
      if (!mbar_wait(&bar_accfull[a], aph, abort_flag, ws, 0x40000u | a)) break;
      tc_fence_after();
      const int ch_base = t.nt * p.n_tile;
      for (int b = 0; b < nblk; ++b) {
        const int m = b * 128 + q * 32 + lane;
        const int yy = m / p.P, xx = m - yy * p.P;
        const bool valid = (m < rows) && (xx < tw_valid) && (yy < t.th);
        const size_t pix = ((size_t)t.img * p.ho + (t.y0 + yy)) * p.wo + (x0 + xx);
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * (uint32_t)p.acc_cols + (uint32_t)(b * p.n_tile);
        for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
          if (ch_base + c0 >= p.c_out) break;    // uniform across the warp
          uint32_t v[16];
          tmem_ld16(taddr + (uint32_t)c0, v);
          tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int hlf = 0; hlf < 2; ++hlf) {
              const int ch = ch_base + c0 + hlf * 8;
              if (ch < p.c_out) {
                float f[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[hlf * 8 + i]);
                if (bias) {
                  const float4 b0 = *reinterpret_cast<const float4 *>(bias + ch);
                  const float4 b1 = *reinterpret_cast<const float4 *>(bias + ch + 4);
                  f[0] += b0.x; f[1] += b0.y; f[2] += b0.z; f[3] += b0.w;
                  f[4] += b1.x; f[5] += b1.y; f[6] += b1.z; f[7] += b1.w;
                }
                if (residual) {
                  const uint4 rv = *reinterpret_cast<const uint4 *>(residual + pix * p.c_out + ch);
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
                *reinterpret_cast<uint4 *>(y + pix * p.c_out + ch) = ov;
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&bar_accempty[a]);
    }
  }

  // ---- teardown.  After a timeout, give copies and MMAs still in flight time to land before
  // shared and tensor memory are released.
  if (*abort_flag) {
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
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

// Chooses tiles, stages and the launch shape; false when the shape is outside this kernel's range.
bool tc_plan(int n, int h, int w, const dc_geom *g, int n_sm, TcParams *p) {
  if (g->groups != 1 || g->c_in % 8 || g->c_out % 8) return false;
  if (g->stride != 1 && g->stride != 2) return false;
  if (g->k > 7) return false;
  if (g->stride == 2 && (w % 2 || g->k == 1)) return false;
  KOrder ko;
  dc_korder_init(&ko, g);
  if (ko.e_pad > 256) return false;
  const int ho = dc_out_extent(h, g->k, g->stride, g->pad), wo = dc_out_extent(w, g->k, g->stride, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  if ((long long)n * h * w * g->c_in >= (1ll << 40)) return false;
  const bool flat = (g->k == 1 && g->stride == 1 && g->pad == 0);

  p->ko = ko;
  p->stride = g->stride;
  p->c_out = g->c_out;
  p->cg = ko.cg; p->ng = ko.ng; p->e_pad = ko.e_pad; p->cch = ko.cch; p->pcs = ko.pcs;
  p->nnt = dc_div_up(ko.n_pad, 256);
  p->n_tile = (int)dc_round_up((size_t)dc_div_up(ko.n_pad, p->nnt), 16);
  int mb_max = 256 / p->n_tile;
  if (mb_max > 8) mb_max = 8;
  if (mb_max < 1) return false;
  p->b_stage_bytes = ko.e_pad * p->n_tile * 16;
  p->b_resident = (ko.ng == 1 && p->nnt == 1) ? 1 : 0;

  if (flat) {
    long long pixels = (long long)n * h * w;
    if (pixels >= (1ll << 31)) return false;
    p->n_img = 1; p->h = 1; p->w = (int)pixels; p->ho = 1; p->wo = (int)pixels;
    int mbf = mb_max < 2 ? mb_max : 2;
    // keep at least ~4 tiles per SM when the map is small
    while (mbf > 1 && pixels / (128 * mbf) < 4ll * n_sm) --mbf;
    p->tw = 128 * mbf; p->th = 1;
    p->wbox = p->tw; p->rbox = 1;
    p->P = p->tw;
    p->cx0 = 0; p->cy0 = 0;
  } else {
    p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
    const int halo_lo = (g->stride == 1) ? 0 : 0;
    (void)halo_lo;
    int nxt = dc_div_up(wo, 64);
    p->tw = dc_div_up(wo, nxt);
    if (g->stride == 1) {
      p->wbox = p->tw + g->k - 1;
      p->P = p->wbox;
      p->cx0 = -g->pad; p->cy0 = -g->pad;
    } else {
      p->wbox = p->tw + dc_floor_div2(g->k - 1 - g->pad) - dc_floor_div2(-g->pad);
      p->P = 2 * p->wbox;
      p->cx0 = dc_floor_div2(-g->pad); p->cy0 = -g->pad;
    }
    if (p->wbox > 256) return false;
    // rows per tile: bounded by the accumulator blocks, the image, shared memory, and a target
    // of about six tiles per CTA so that load, MMA and epilogue overlap
    long long total_rows = (long long)n * ho * dc_div_up(wo, p->tw) * p->nnt;
    int th_target = (int)(total_rows / ((long long)n_sm * 6));
    if (th_target < 1) th_target = 1;
    int th = (mb_max * 128 - p->tw) / p->P + 1;
    if (th < 1) return false;
    if (th > ho) th = ho;
    if (th > th_target) th = th_target;
    for (;; --th) {
      if (th < 1) return false;
      int rbox = (g->stride == 1) ? th + g->k - 1 : 2 * (th - 1) + g->k;
      long long stage = (long long)ko.pcs * ko.cg * rbox * p->wbox * 16;
      if (rbox <= 256 && stage <= 56 * 1024) { p->rbox = rbox; break; }
    }
    p->th = th;
  }
  p->nxt = dc_div_up(p->wo, p->tw);
  p->mb = dc_div_up((p->th - 1) * p->P + p->tw, 128);
  if (p->mb > mb_max) return false;
  p->plane_bytes = p->rbox * p->wbox * 16;
  p->region_bytes = (int)dc_round_up((size_t)ko.cg * p->plane_bytes + 16, 128);
  p->a_stage_bytes = ko.pcs * p->region_bytes;
  p->acc_cols = p->mb * p->n_tile;
  int cols = 32;
  while (cols < 2 * p->acc_cols) cols *= 2;
  if (cols > 512) return false;
  p->tmem_cols = cols;
  long long units = (long long)p->n_img * p->nxt * p->ho;
  if (units * p->nnt >= (1ll << 31)) return false;
  p->units_per_nt = (int)units;
  p->total_units = (int)(units * p->nnt);

  // stages: as many as fit (2..kMaxStages), no more than a CTA will ever use
  const int slack = p->mb * 2048 + 1024;
  int stages = kMaxStages;
  for (;; --stages) {
    if (stages < 2) return false;
    long long tot = 1024ll + (long long)(p->b_resident ? 1 : stages) * p->b_stage_bytes +
                    (long long)stages * p->a_stage_bytes + slack;
    if (tot <= kSmemBudget) { p->smem_bytes = (int)tot; break; }
  }
  p->stages = stages;
  return true;
}

}  // namespace

bool dc_conv_tc_supported(int n, int h, int w, const dc_geom *g) {
  TcParams p;
  return tc_plan(n, h, w, g, 148, &p);
}

dc_status dc_launch_conv_tc(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                            const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                            cudaStream_t stream) {
  TcParams p;
  const int n_sm = sm_count();
  if (!tc_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return DC_ERR_CUDA;

  CUtensorMap map_a, map_b;
  {
    const cuuint64_t C2 = (cuuint64_t)g->c_in * 2;
    cuuint64_t gdim[5], gstr[4];
    if (p.stride == 1) {
      gdim[0] = 8; gdim[1] = (cuuint64_t)p.w; gdim[2] = (cuuint64_t)p.h; gdim[3] = (cuuint64_t)p.n_img;
      gdim[4] = (cuuint64_t)p.cch;
      gstr[0] = C2; gstr[1] = C2 * p.w; gstr[2] = C2 * p.w * p.h; gstr[3] = 16;
    } else {
      gdim[0] = 8; gdim[1] = (cuuint64_t)p.w / 2; gdim[2] = (cuuint64_t)p.h; gdim[3] = (cuuint64_t)p.n_img;
      gdim[4] = (cuuint64_t)2 * p.cch;
      gstr[0] = 2 * C2; gstr[1] = C2 * p.w; gstr[2] = C2 * p.w * p.h; gstr[3] = 16;
    }
    cuuint32_t box[5] = {8, (cuuint32_t)p.wbox, (cuuint32_t)p.rbox, 1, (cuuint32_t)p.cg};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    CUresult r = encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(x), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  {
    cuuint64_t gdim[3] = {8, (cuuint64_t)p.ko.n_pad, (cuuint64_t)p.ng * p.e_pad};
    cuuint64_t gstr[2] = {16, (cuuint64_t)p.ko.n_pad * 16};
    cuuint32_t box[3] = {8, (cuuint32_t)p.n_tile, (cuuint32_t)p.e_pad};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(w_packed), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  static bool attr_set = false;
  if (!attr_set) {
    DC_CUDA_OK(cudaFuncSetAttribute(k_conv_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    attr_set = true;
  }
  int grid = p.total_units < n_sm ? p.total_units : n_sm;
  k_conv_tc<<<grid, kThreads, p.smem_bytes, stream>>>(map_a, map_b, p, bias, (const __nv_bfloat16 *)residual,
                                                     (__nv_bfloat16 *)y, (DcWsHeader *)workspace);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
