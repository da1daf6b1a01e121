// Dense convolution forward as an implicit GEMM on the 5th-generation tensor cores (sm_100a):
// tcgen05.mma with the accumulator in tensor memory, operands staged in shared memory.
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
// Stride 2 splits the patch by input-column parity (two sets of planes at half resolution) and, inside
// a plane, by row parity (even patch rows first): a tap then reads consecutive rows for consecutive
// output rows, and the GEMM rows enumerate output pixels only.
//
// One tensor-core instruction takes K = 16 = two 16-byte chunks, addressed as "start" and
// "start + LBO": any two chunk entries whose addresses increase can be paired, which is how
// channel counts that are not multiples of 16 (24 = 3 chunks) avoid padding.
//
// Staging.  Activations: four producer warps gather the patch with 16-byte cp.async copies
// (global reads of a warp are contiguous; the scatter into planes happens on the shared-memory
// side; halo pixels are zero-filled).  A tiled TMA copy cannot produce this layout at speed: its
// innermost box row would be 16 bytes, and one request per 16 bytes measured 27 us for a 19 MB
// problem.  Weights: the packed layout in HBM is the operand layout, so a (channel group, output-
// channel pass) tile is one contiguous bulk copy (cp.async.bulk; one per entry when the output
// channels are cut into passes), resident for the whole kernel when it fits.  Output: the epilogue converts to bf16 into a dense shared-memory
// tile and one bulk copy (cp.async.bulk shared -> global) writes it when the tile is contiguous
// in global memory; otherwise 16-byte stores.
//
// Roles per CTA (288 threads): warps 0-3 producers, warp 4 lane 0 issues the MMAs and warp 4
// owns the tensor-memory allocation, warps 5-8 epilogue.  Accumulators are double buffered so the
// epilogue of tile i overlaps the MMAs of tile i+1.  Every wait is bounded: when one runs out the
// CTA latches DC_ERR_TIMEOUT in the caller's workspace and leaves.
#include <type_traits>
#include "tc_ptx.cuh"

namespace {

constexpr int kMaxStages = 8;
constexpr int kProducerThreads = 128;
constexpr int kThreads = 288;
constexpr int kMaxPieces = 16;          // 16-byte pieces of one patch row handled by one producer thread

struct TcParams {
  int n_img, h, w, ho, wo, c_in, c_out;
  int k, stride;
  int tw, th, nxt;            // tile width / height in outputs, x tiles per row
  int P, mb;                  // GEMM-row pitch per output row, 128-row blocks per tile
  int n_tile, nnt;            // output channels per pass, passes
  int units_per_nt, total_units;
  int cg, ng, e_pad, cch, pcs;
  int wbox, rbox;             // patch columns (per parity), rows
  int odd_rows_off;           // stride 2: byte offset of the odd patch rows inside a plane (even rows come first)
  int plane_stride, region_bytes, a_stage_bytes, b_stage_bytes;
  int stages, b_resident;
  int act;
  int cx0, cy0;               // patch origin: x = xt*tw + cx0 (parity-plane columns), y = y0*stride + cy0
  int acc_cols, tmem_cols;
  int acc_slots;              // accumulator sets in tensor memory: 2 (epilogue of a tile under the next tile's MMAs) or 1
  int bulk_out, out_tile_bytes;
  int off_b, off_a, off_out, off_bias;  // offsets in dynamic shared memory
  int smem_bytes;
  KOrder ko;
  // per instruction j: low word of its A descriptor relative to the stage base:
  // (offset of first chunk >> 4) | (distance to second chunk >> 4) << 16.  Lives in the kernel
  // parameters (constant bank) so that the issuing warp reads it with uniform loads.
  uint32_t a_desc_lo[128];
};

using namespace tc;

// ------------------------------------------------------------------------------------------ tiles
struct Tile {
  int nt, img, xt, y0, th;
};

// Units are output row segments ordered (nt, img, xt, y); a CTA owns a contiguous range of them
// and cuts it into tiles of up to p.th rows that never cross an image or column-strip boundary.
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
k_conv_tc(const void *__restrict__ w_packed, const __grid_constant__ TcParams p,
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
  uint8_t *smem_zero = smem_a + (size_t)p.stages * p.a_stage_bytes;   // always-zero plane + slack
  uint8_t *smem_ones = smem + p.off_bias;        // 8 GEMM rows of the constant operand: (1, 1, 0, ..) in 16 bytes each
  uint8_t *smem_bias = smem_ones + 128;          // [nnt * n_tile][16 bytes]: bias as two bf16 terms, then n_tile zero rows

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t *abort_flag = &abort_s;
  const bool odd_entries = (p.ko.e & 1) != 0;

  // ---- set-up
  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < p.stages; ++s) { mbar_init(&bar_full[s], kProducerThreads); mbar_init(&bar_empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bar_accfull[a], 1); mbar_init(&bar_accempty[a], 128); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Nothing above touched global memory; everything below may.  Tensor memory is allocated after this
  // point on purpose: a CTA that held columns while it waits here for the previous kernel could keep a
  // CTA of that kernel on the same SM from getting its own.
  dc_pdl_enter();
  if (warp == 4) {
    tmem_alloc(&tmem_base_s, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  if (threadIdx.x >= 5 * 32) {
    const int t = threadIdx.x - 5 * 32;
    // The bias is added by the tensor core: one instruction per block multiplies a constant operand (1.0 in
    // the first two K elements of every GEMM row; one 8-row group read sixteen times, group stride 0; its
    // second K chunk is the zero plane) with [bias as bf16, its bf16 remainder, 0, ...] per output channel
    // (exact to 16 mantissa bits) before the block's other instructions accumulate.
    if (t < 8) reinterpret_cast<uint4 *>(smem_ones)[t] = make_uint4(0x3F803F80u, 0u, 0u, 0u);
    for (int i = t; i < (p.nnt + 1) * p.n_tile; i += 128) {
      uint32_t w0 = 0u;
      if (bias && i < p.c_out) {
        const float b = bias[i];
        const __nv_bfloat16 hi = __float2bfloat16_rn(b);
        const __nv_bfloat16 lo = __float2bfloat16_rn(b - __bfloat162float(hi));
        w0 = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16);
      }
      reinterpret_cast<uint4 *>(smem_bias)[i] = make_uint4(w0, 0u, 0u, 0u);
    }
    // the zero plane: second chunk of the padding entry, and the landing zone of reads past the last stage
    uint4 *z = reinterpret_cast<uint4 *>(smem_zero);
    for (int i = t; i < (p.mb * 2048 + 1024) / 16; i += 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  const int cta_begin = (int)((long long)p.total_units * blockIdx.x / gridDim.x);
  const int cta_end = (int)((long long)p.total_units * (blockIdx.x + 1) / gridDim.x);

  if (warp < 4) {
    // ================================================================== producers (cp.async, bulk copies for weights)
    const int ptid = threadIdx.x;
    const int row_pieces = p.wbox * p.pcs * p.cg;
    const int C2 = p.c_in * 2;
    const int npieces = (ptid < row_pieces) ? (row_pieces - ptid + kProducerThreads - 1) / kProducerThreads : 0;
    int src_off[kMaxPieces], gx_rel[kMaxPieces];
    uint32_t dst_off[kMaxPieces];
#pragma unroll
    for (int i = 0; i < kMaxPieces; ++i) {
      if (i >= npieces) break;
      const int q = ptid + i * kProducerThreads;
      const int ccg = q % p.cg;
      const int t = q / p.cg;
      const int pc = t % p.pcs;
      const int col = t / p.pcs;
      gx_rel[i] = (p.stride == 1) ? col : 2 * col + pc;
      src_off[i] = gx_rel[i] * C2 + ccg * 16;
      dst_off[i] = (uint32_t)(pc * p.region_bytes + ccg * p.plane_stride + col * 16);
    }
    const uint32_t a_base0 = smem_u32(smem_a);
    const long long row_stride = (long long)p.w * C2;
    const uint32_t drow_stride = (uint32_t)p.wbox * 16u;
    uint32_t it = 0;
    bool b_loaded = false, ok = true;
    for (int cur = cta_begin; cur < cta_end && ok;) {
      const Tile t = decode_tile(p, cur, cta_end);
      cur += t.th;
      const int gx0 = (t.xt * p.tw + p.cx0) * p.stride;
      const int gy0 = t.y0 * p.stride + p.cy0;
      const int rows = (t.th - 1) * p.stride + p.k;
      const int r_lo = gy0 < 0 ? -gy0 : 0;                       // patch rows [r_lo, r_hi) lie inside the image
      const int r_hi = (p.h - gy0 < rows) ? p.h - gy0 : rows;
      const char *tile_base = reinterpret_cast<const char *>(x) + (size_t)t.img * p.h * row_stride +
                              ((long long)gy0 * p.w + gx0) * C2;
      for (int grp = 0; grp < p.ng; ++grp, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!mbar_wait(&bar_empty[s], ph ^ 1, abort_flag, ws, 0x10000u | s)) { ok = false; break; }
        if (ptid == 0) {
          // a weight tile rides along on the same barrier as transaction bytes
          const bool load_b = !p.b_resident || !b_loaded;
          if (load_b) {
            // The packed weights are stored as the operand wants them ([entry][n_pad rows][8]): a
            // group's tile is one contiguous bulk copy, or one per entry when the output channels
            // are cut into passes.  (A tiled TMA load with this 16-byte inner box fetched 16 bytes
            // per request and took microseconds.)
            const uint32_t dst = smem_u32(smem_b + (size_t)(p.b_resident ? 0 : s) * p.b_stage_bytes);
            const char *src = reinterpret_cast<const char *>(w_packed) + (size_t)grp * p.e_pad * p.ko.n_pad * 16;
            if (p.n_tile == p.ko.n_pad) {
              mbar_expect_tx(&bar_full[s], (uint32_t)p.b_stage_bytes);
              bulk_load(dst, src, (uint32_t)p.b_stage_bytes, &bar_full[s]);
            } else {
              const int lo = t.nt * p.n_tile;
              const int rows = (p.ko.n_pad - lo < p.n_tile) ? p.ko.n_pad - lo : p.n_tile;
              mbar_expect_tx(&bar_full[s], (uint32_t)(p.e_pad * rows * 16));
              for (int e = 0; e < p.e_pad; ++e)
                bulk_load(dst + (uint32_t)(e * p.n_tile * 16), src + ((size_t)e * p.ko.n_pad + lo) * 16,
                          (uint32_t)(rows * 16), &bar_full[s]);
            }
            b_loaded = true;
          }
        }
        const uint32_t stage = a_base0 + (uint32_t)s * p.a_stage_bytes;
        const char *grp_base = tile_base + grp * p.cg * 16;
#pragma unroll
        for (int i = 0; i < kMaxPieces; ++i) {
          if (i >= npieces) break;
          const int gx = gx0 + gx_rel[i];
          const bool cv = (gx >= 0) && (gx < p.w);
          const char *src = grp_base + src_off[i];
          // stride 2: the even patch rows of a plane come first, then the odd ones, so that the rows one
          // tap reads for consecutive output rows are consecutive
          uint32_t dst = stage + dst_off[i];
          if (p.stride == 1) {
            for (int r = 0; r < rows; ++r) {
              const bool v = cv && (r >= r_lo) && (r < r_hi);
              cp_async16(dst, v ? (const void *)src : (const void *)x, v ? 16u : 0u);
              src += row_stride;
              dst += drow_stride;
            }
          } else {
            uint32_t dst_odd = dst + (uint32_t)p.odd_rows_off;
            for (int r = 0; r < rows; r += 2) {
              const bool v0 = cv && (r >= r_lo) && (r < r_hi), v1 = cv && (r + 1 >= r_lo) && (r + 1 < r_hi);
              cp_async16(dst, v0 ? (const void *)src : (const void *)x, v0 ? 16u : 0u);
              if (r + 1 < rows) cp_async16(dst_odd, v1 ? (const void *)(src + row_stride) : (const void *)x, v1 ? 16u : 0u);
              src += 2 * row_stride;
              dst += drow_stride;
              dst_odd += drow_stride;
            }
          }
        }
        cp_async_arrive(&bar_full[s]);           // arrives by itself when this thread's copies have landed
      }
    }
    cp_async_wait_all();                         // nothing of this thread is in flight when the CTA leaves
  } else if (warp == 4) {
    // ================================================================== MMA issuer
    // The whole warp walks the loop converged and one elected lane issues: every operand is then
    // warp-uniform (kernel parameters and loop counters), which keeps descriptor arithmetic cheap.
    {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_tile >> 3) << 17) | (8u << 24);
      const uint32_t desc_hi = (128u >> 4) | (1u << 14);
      const int npairs = p.e_pad / 2;
      const uint32_t zero_addr = smem_u32(smem_zero);
      // one election for the whole role: the same lane issues every instruction, a stage's instructions in one
      // stretch (an election and a branch per instruction cost the warp several times the instruction itself)
      const bool leader = elect_one();
      uint32_t it = 0, tile_i = 0;
      for (int cur = cta_begin; cur < cta_end; ++tile_i) {
        const Tile t = decode_tile(p, cur, cta_end);
        cur += t.th;
        const int rows = (t.th - 1) * p.P + p.tw;
        const int nblk = (rows + 127) >> 7;
        const uint32_t a = p.acc_slots == 2 ? (tile_i & 1) : 0u, aph = p.acc_slots == 2 ? ((tile_i >> 1) & 1) : (tile_i & 1);
        if (!warp_wait(&bar_accempty[a], aph ^ 1, abort_flag, ws, 0x20000u | a)) goto mma_done;
        tc_fence_after();
        const uint32_t d0 = tmem_base + a * (uint32_t)p.acc_cols;
        {
          // the bias initialises the accumulators of the tile's blocks (it needs no load)
          const uint32_t ones_a = smem_u32(smem_ones), bias_a = smem_u32(smem_bias) + (uint32_t)(t.nt * p.n_tile * 16);
          const uint32_t zero_rows = smem_u32(smem_bias) + (uint32_t)(p.nnt * p.n_tile * 16);
          const uint64_t ad = ((uint64_t)(1u << 14) << 32) | (uint64_t)(((ones_a >> 4) & 0x3FFFu) | (((zero_addr - ones_a) >> 4) << 16));
          const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(((bias_a >> 4) & 0x3FFFu) | (((zero_rows - bias_a) >> 4) << 16));
          if (leader)
            for (int b = 0; b < nblk; ++b) umma_bf16(d0 + (uint32_t)(b * p.n_tile), ad, bd, idesc, 0u);
          __syncwarp();
        }
        for (int grp = 0; grp < p.ng; ++grp, ++it) {
          const int s = it % p.stages;
          const uint32_t ph = (it / p.stages) & 1;
          if (!warp_wait(&bar_full[s], ph, abort_flag, ws, 0x30000u | s)) goto mma_done;
          fence_proxy_async();
          tc_fence_after();
          const uint32_t a_base = smem_u32(smem_a + (size_t)s * p.a_stage_bytes);
          const uint32_t b_base = smem_u32(smem_b + (size_t)(p.b_resident ? 0 : s) * p.b_stage_bytes);
          const uint32_t b_lo0 = ((b_base >> 4) & 0x3FFFu) | ((uint32_t)p.n_tile << 16);
          const uint32_t b_step = 2u * (uint32_t)p.n_tile;
          // last pair of an odd entry count: second chunk = zero plane (same block offset on both sides)
          const uint32_t last = (uint32_t)(npairs - 1);
          const uint32_t first_off = (p.a_desc_lo[last] & 0x3FFFu) << 4;
          const uint32_t pad_lo = (first_off >> 4) | (((zero_addr - a_base - first_off) >> 4) << 16);
          if (leader) {
            for (int b = 0; b < nblk; ++b) {
              const uint32_t d = d0 + (uint32_t)(b * p.n_tile);
              const uint32_t a_add = (a_base >> 4) + (uint32_t)b * 128u;
#pragma unroll 4
              for (int j = 0; j < npairs; ++j) {
                uint32_t lo = p.a_desc_lo[j];
                if (odd_entries && (uint32_t)j == last) lo = pad_lo;
                const uint64_t ad = ((uint64_t)desc_hi << 32) | (uint64_t)(lo + a_add);
                const uint64_t bd = ((uint64_t)desc_hi << 32) | (uint64_t)(b_lo0 + (uint32_t)j * b_step);
                umma_bf16(d, ad, bd, idesc, 1u);
              }
            }
            umma_commit(&bar_empty[s]);          // stage s may be refilled once these MMAs finish
          }
          __syncwarp();
        }
        if (leader) umma_commit(&bar_accfull[a]);        // accumulator a is complete
        __syncwarp();
      }
    }
  mma_done:;
  } else {
    // ================================================================== epilogue (4 warps)
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    const bool elected = (threadIdx.x == 5 * 32);
    uint32_t tile_i = 0;
    for (int cur = cta_begin; cur < cta_end; ++tile_i) {
      const Tile t = decode_tile(p, cur, cta_end);
      cur += t.th;
      const int rows = (t.th - 1) * p.P + p.tw;
      const int nblk = (rows + 127) >> 7;
      const int x0 = t.xt * p.tw;
      const int tw_valid = (p.wo - x0 < p.tw) ? p.wo - x0 : p.tw;
      const uint32_t a = p.acc_slots == 2 ? (tile_i & 1) : 0u, aph = p.acc_slots == 2 ? ((tile_i >> 1) & 1) : (tile_i & 1);
      uint8_t *obuf = smem_out + (size_t)(tile_i & 1) * p.out_tile_bytes;
      if (p.bulk_out && elected) bulk_wait_read1();   // the store that last used this buffer has read it
      // all 128 epilogue threads pass or leave together, so nobody is left alone at a named barrier
      if (!epi_all(mbar_wait(&bar_accfull[a], aph, abort_flag, ws, 0x40000u | a))) break;
      tc_fence_after();
      const int ch_base = t.nt * p.n_tile;
      for (int b = 0; b < nblk; ++b) {
        const int m = b * 128 + q * 32 + lane;
        const int yy = m / p.P, xx = m - yy * p.P;
        const bool valid = (m < rows) && (xx < tw_valid) && (yy < t.th);
        const size_t pix = ((size_t)t.img * p.ho + (t.y0 + yy)) * p.wo + (x0 + xx);
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * (uint32_t)p.acc_cols + (uint32_t)(b * p.n_tile);
        __nv_bfloat16 *gout = y + pix * p.c_out;
        const __nv_bfloat16 *gres = residual ? residual + pix * p.c_out : nullptr;
        uint8_t *sout = obuf + (size_t)(yy * p.tw + xx) * p.c_out * 2;
        // activation and skip input are compile-time in the per-pixel code (four instantiations, picked once
        // per block); the pixel goes to the staged tile or straight to memory through one generic pointer
        uint8_t *const pdst = p.bulk_out ? sout : reinterpret_cast<uint8_t *>(gout);
        auto channels = [&](auto RELU, auto RES) {
          for (int c0 = 0; c0 < p.n_tile; c0 += 32) {
            if (ch_base + c0 >= p.c_out) break;    // uniform across the warp
            uint32_t v[32];
            const bool wide = (c0 + 32 <= p.n_tile);
            if (wide) tmem_ld32(taddr + (uint32_t)c0, v);
            else tmem_ld16(taddr + (uint32_t)c0, v);
            tmem_ld_wait();
            if (valid) {
#pragma unroll
              for (int e8 = 0; e8 < 4; ++e8) {
                const int ch = ch_base + c0 + e8 * 8;
                if ((e8 < 2 || wide) && ch < p.c_out) {
                  float f[8];                      // the bias is in the accumulator already
#pragma unroll
                  for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[e8 * 8 + i]);
                  if (decltype(RES)::value) {
                    const uint4 rv = *reinterpret_cast<const uint4 *>(gres + ch);
                    const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                      const float2 rf = __bfloat1622float2(rb[i]);
                      f[2 * i] += rf.x; f[2 * i + 1] += rf.y;
                    }
                  }
                  uint4 ov;
                  uint32_t *ow = reinterpret_cast<uint32_t *>(&ov);
                  // ReLU6: the conversion clamps at zero itself, one packed minimum against (6, 6) does the rest
                  // (the same values as clamping before rounding, since 0 and 6 are bf16 values)
#pragma unroll
                  for (int i = 0; i < 4; ++i)
                    ow[i] = decltype(RELU)::value ? min_bf16x2(pack_bf16x2_relu(f[2 * i], f[2 * i + 1]), 0x40C040C0u)
                                                  : pack_bf16x2(f[2 * i], f[2 * i + 1]);
                  *reinterpret_cast<uint4 *>(pdst + ch * 2) = ov;
                }
              }
            }
          }
        };
        using T = std::true_type;
        using F = std::false_type;
        if (p.act == DC_ACT_RELU6) { if (gres) channels(T{}, T{}); else channels(T{}, F{}); }
        else { if (gres) channels(F{}, T{}); else channels(F{}, F{}); }
      }
      tc_fence_before();
      mbar_arrive(&bar_accempty[a]);
      if (p.bulk_out) {
        fence_proxy_async();                     // the tile written above is read by the bulk copy engine
        epi_barrier();
        if (elected) {
          const size_t pix0 = ((size_t)t.img * p.ho + t.y0) * p.wo + x0;
          const uint32_t bytes = (uint32_t)(((p.ho == 1) ? tw_valid : t.th * p.tw) * p.c_out * 2);
          bulk_store(y + pix0 * p.c_out, smem_u32(obuf), bytes);
          bulk_commit();
        }
      }
    }
    if (p.bulk_out && elected) bulk_wait_all();
  }

  // ---- teardown.  After a timeout, give copies and MMAs still in flight time to land before
  // shared and tensor memory are released.
  if (*abort_flag) {
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// ------------------------------------------------------------------------------------------ host
constexpr int kSmemBudget = 200 * 1024;

// plane stride in 16-byte units is made congruent to `want` mod 8 so that the cg chunks of one
// pixel, written by neighbouring producer threads, fall into different bank groups
int padded_plane_units(int units, int cg) {
  int want = (cg == 3 || cg == 5 || cg == 7) ? cg : (cg >= 8 ? 1 : (8 / cg));
  while ((units & 7) != (want & 7)) ++units;
  return units;
}

// Chooses tiles, stages and the launch shape; false when the shape is outside this kernel's range.
bool tc_plan(int n, int h, int w, const dc_geom *g, int n_sm, TcParams *p) {
  if (g->groups != 1 || g->c_in % 8 || g->c_out % 8) return false;
  if (g->stride != 1 && g->stride != 2) return false;
  if (g->k > 7) return false;
  if (g->stride == 2 && (w % 2 || g->k == 1)) return false;
  KOrder ko;
  dc_korder_init(&ko, g);
  if (ko.e_pad > 256 || ko.fold || ko.pair || ko.rows) return false;    // fold- and pair-order weights belong to their own kernels
  const int ho = dc_out_extent(h, g->k, g->stride, g->pad), wo = dc_out_extent(w, g->k, g->stride, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  if ((long long)n * h * w * g->c_in >= (1ll << 40)) return false;
  const bool flat = (g->k == 1 && g->stride == 1 && g->pad == 0);

  p->ko = ko;
  p->k = g->k;
  p->stride = g->stride;
  p->c_in = g->c_in;
  p->c_out = g->c_out;
  p->cg = ko.cg; p->ng = ko.ng; p->e_pad = ko.e_pad; p->cch = ko.cch; p->pcs = ko.pcs;
  p->nnt = dc_div_up(ko.n_pad, 256);
  p->n_tile = (int)dc_round_up((size_t)dc_div_up(ko.n_pad, p->nnt), 16);
  p->b_stage_bytes = ko.e_pad * p->n_tile * 16;
  p->b_resident = (ko.ng == 1 && p->nnt == 1) ? 1 : 0;
  // Two accumulator sets let the epilogue of a tile run under the next tile's MMAs.  Wide outputs leave
  // room for one 128-row block per set only; when the weights are streamed per (tile, channel group)
  // as well, one set of up to three blocks is better: a weight stage then serves three times the rows.
  int mb_max = 256 / p->n_tile;
  p->acc_slots = 2;
  if (mb_max < 2 && !p->b_resident && 512 / p->n_tile >= 2) {
    p->acc_slots = 1;
    mb_max = 512 / p->n_tile;
  }
  if (mb_max > 8) mb_max = 8;
  if (mb_max < 1) return false;

  if (flat) {
    long long pixels = (long long)n * h * w;
    if (pixels >= (1ll << 31)) return false;
    p->n_img = 1; p->h = 1; p->w = (int)pixels; p->ho = 1; p->wo = (int)pixels;
    int mbf = mb_max < 2 ? mb_max : 2;
    while (mbf > 1 && pixels / (128 * mbf) < 4ll * n_sm) --mbf;     // keep several tiles per SM
    p->tw = 128 * mbf; p->th = 1;
    p->wbox = p->tw; p->rbox = 1;
    p->P = p->tw;
    p->cx0 = 0; p->cy0 = 0;
  } else {
    p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
    int nxt = dc_div_up(wo, 64);
    p->tw = dc_div_up(wo, nxt);
    if (g->stride == 1) {
      p->wbox = p->tw + g->k - 1;
      p->P = p->wbox;
      p->cx0 = -g->pad; p->cy0 = -g->pad;
    } else {
      p->wbox = p->tw + dc_floor_div2(g->k - 1 - g->pad) - dc_floor_div2(-g->pad);
      p->P = p->wbox;
      p->cx0 = dc_floor_div2(-g->pad); p->cy0 = -g->pad;
    }
    // rows per tile: bounded by the accumulator blocks, the image, shared memory, and a target
    // of about six tiles per CTA so that load, MMA and epilogue overlap
    long long total_rows = (long long)n * ho * dc_div_up(wo, p->tw) * p->nnt;
    int th_target = (int)(total_rows / ((long long)n_sm * (p->acc_slots == 2 ? 6 : 2)));
    if (th_target < 1) th_target = 1;
    int th = (mb_max * 128 - p->tw) / p->P + 1;
    if (th < 1) return false;
    if (th > ho) th = ho;
    if (th > th_target) th = th_target;
    for (;; --th) {
      if (th < 1) return false;
      int rbox = (g->stride == 1) ? th + g->k - 1 : 2 * (th - 1) + g->k;
      long long stage = (long long)ko.pcs * ko.cg * (rbox * p->wbox + 8) * 16;
      if (stage <= 56 * 1024) { p->rbox = rbox; break; }
    }
    p->th = th;
  }
  if (p->wbox * p->pcs * p->cg > kMaxPieces * kProducerThreads) return false;
  p->nxt = dc_div_up(p->wo, p->tw);
  p->mb = dc_div_up((p->th - 1) * p->P + p->tw, 128);
  if (p->mb > mb_max) return false;
  p->odd_rows_off = (g->stride == 2) ? ((p->rbox + 1) / 2) * p->wbox * 16 : 0;
  p->plane_stride = padded_plane_units(p->rbox * p->wbox + 1, ko.cg) * 16;
  p->region_bytes = (int)dc_round_up((size_t)ko.cg * p->plane_stride, 128);
  p->a_stage_bytes = ko.pcs * p->region_bytes;
  p->acc_cols = p->mb * p->n_tile;
  int cols = 32;
  while (cols < p->acc_slots * p->acc_cols) cols *= 2;
  if (cols > 512) return false;
  p->tmem_cols = cols;
  long long units = (long long)p->n_img * p->nxt * p->ho;
  if (units * p->nnt >= (1ll << 31)) return false;
  p->units_per_nt = (int)units;
  p->total_units = (int)(units * p->nnt);

  // output staging: one bulk copy per tile when the tile is contiguous in global memory
  p->out_tile_bytes = (int)dc_round_up((size_t)p->th * p->tw * g->c_out * 2, 128);
  p->bulk_out = (p->nnt == 1 && (flat || p->tw == p->wo) && p->out_tile_bytes <= 24 * 1024) ? 1 : 0;
  if (!p->bulk_out) p->out_tile_bytes = 0;

  // shared memory: [weights][bias][output tiles x2][activation stages][slack]
  const int slack = p->mb * 2048 + 1024;
  const int bias_bytes = (int)dc_round_up((size_t)128 + (size_t)(p->nnt + 1) * p->n_tile * 16, 128);   // constant operand, bias rows, zero rows
  int stages = kMaxStages;
  for (;; --stages) {
    if (stages < 2) return false;
    long long tot = 1024ll + (long long)(p->b_resident ? 1 : stages) * p->b_stage_bytes + bias_bytes +
                    2ll * p->out_tile_bytes + (long long)stages * p->a_stage_bytes + slack;
    if (tot <= kSmemBudget) { p->smem_bytes = (int)tot; break; }
  }
  // no point in more stages than a CTA has (tile, group) pairs
  long long per_cta = ((long long)p->total_units / p->th / n_sm + 2) * p->ng;
  if (stages > per_cta) stages = (int)per_cta;
  if (stages < 2) stages = 2;
  p->stages = stages;
  p->off_b = 0;
  p->off_bias = (p->b_resident ? 1 : stages) * p->b_stage_bytes;
  p->off_out = p->off_bias + bias_bytes;
  p->off_a = p->off_out + 2 * p->out_tile_bytes;
  p->smem_bytes = 1024 + p->off_a + stages * p->a_stage_bytes + slack;
  // chunk-pair table: entry e -> byte offset of its 16-byte column in an A stage.  The padding
  // entry of an odd count gets its distance at issue time (it points at the zero plane).
  for (int j = 0; j < ko.e_pad / 2; ++j) {
    uint32_t off[2] = {0u, 16u};
    for (int q = 0; q < 2; ++q) {
      int pc, ccg, r, s;
      if (dc_korder_decode(ko, 2 * j + q, &pc, &ccg, &r, &s)) {
        int sx = (g->stride == 1) ? s : dc_floor_div2(s - g->pad) - dc_floor_div2(-g->pad);
        const int row = (g->stride == 1) ? r : (r >> 1);       // stride 2: row r / 2 of the rows of r's parity
        off[q] = (uint32_t)(pc * p->region_bytes + ccg * p->plane_stride + (r & (g->stride - 1)) * p->odd_rows_off +
                            (row * p->wbox + sx) * 16);
      } else if (q == 1) {
        off[1] = off[0] + 16;
      }
    }
    // the second chunk is addressed as a 14-bit distance in 16-byte units above the first
    if (off[1] <= off[0] || ((off[1] - off[0]) >> 4) > 0x3FFFu) return false;
    p->a_desc_lo[j] = (off[0] >> 4) | (((off[1] - off[0]) >> 4) << 16);
  }
  return true;
}

}  // namespace

bool dc_conv_tc_supported(int n, int h, int w, const dc_geom *g) {
  TcParams p;
  return tc_plan(n, h, w, g, dc_sm_count(), &p);
}

dc_status dc_launch_conv_tc(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                            const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                            cudaStream_t stream) {
  TcParams p;
  const int n_sm = dc_sm_count();
  if (!tc_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  static unsigned char attr_done[kDcMaxDevices];
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_tc, kSmemBudget, attr_done));
  int grid = p.total_units < n_sm ? p.total_units : n_sm;
  const cudaError_t le = dc_launch_pdl(k_conv_tc, dim3(grid), dim3(kThreads), (size_t)p.smem_bytes, stream, w_packed, p,
                                       (const __nv_bfloat16 *)x, bias, (const __nv_bfloat16 *)residual,
                                       (__nv_bfloat16 *)y, (DcWsHeader *)workspace);
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
