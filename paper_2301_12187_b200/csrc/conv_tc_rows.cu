// Dense stride-1 convolution with many input channels as an implicit GEMM over PIXEL ROWS fed
// straight from TMA tiles (see KOrder, "rows" order).
//
// A shared-memory line (128 bytes) holds 64 channels of one pixel; the input channels are cut into
// planes of 64 (the last one zero filled by the TMA unit), and a GEMM row is a pixel of the haloed
// patch.  Tap (r, s) of plane g is the plane's tile read (r * patch width + s) lines further on, so
// one 4-D TMA load per (tile, plane) -- box 64 channels x patch width x patch rows x images, 128-byte
// swizzle, zero fill outside the image -- feeds every instruction of that plane.  Small feature
// maps are tiled several images at a time (the box's image extent), so that the 128 rows of a
// block are not mostly halo and the weights, which are far larger than the activations in these
// layers, are streamed once per group of images instead of once per image.
//
// The reduction runs over (plane g, tap row r) steps.  Each step needs k * nsl(g) * 2 chunk planes
// of weights ([n_tile rows][8] bf16, no swizzle), which stream through their own ring: a layer such
// as 160 -> 960, 3x3 has 2.8 MB of weights, 40x the activations of an image.  Output channels go in
// passes of n_tile <= 128; accumulators (blocks of 128 rows x n_tile columns) live in tensor memory,
// two sets when they fit so that the epilogue of one work item overlaps the MMAs of the next.
//
// Roles (352 threads): warp 0 producer (issues TMA / bulk loads in consumption order),
// warps 1-2 MMA issue (blocks alternate between them), warps 3-10 epilogue (two per tensor-memory
// lane quadrant, blocks alternate).  A work item is (tile, output-channel pass); CTAs (one per SM)
// take contiguous runs of items.  All waits are bounded (tc::mbar_wait).
#include <type_traits>
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr int kMaxA = 8;                         // activation plane stages
constexpr int kMaxB = 12;                        // weight stages
constexpr int kFirstA = 3, kFirstB = 4;          // depths reached first (weights, then activations), before the rings deepen in turn
constexpr int kMmaWarp = 1;
constexpr int kMmaWarps = 2;
constexpr int kFirstEpiWarp = kMmaWarp + kMmaWarps;
constexpr int kEpiWarps = 8;
constexpr int kConsumerThreads = (kMmaWarps + kEpiWarps) * 32;
constexpr int kThreads = 32 + kConsumerThreads;
constexpr int kBarConsumers = 7;                 // named barrier of all consumer warps
constexpr int kMaxBlocks = 2;                    // 128-row blocks per tile
constexpr int kStagePitch = 64;                  // bytes per pixel in an epilogue warp's turn-around buffer (pieces XOR-swizzled)

struct RowsParams {
  int n_img, h, w, ho, wo, c_in, c_out;
  int k, pad, planes;          // planes of 64 input channels
  int tw, th, nxt, wbox, rbox, ni;   // tile: outputs per row, rows, strips per row, patch width / rows, images
  int tiles_y, img_groups;
  int grid, items_per, items_rem;    // CTAs; CTA b takes items_per (+1 if b < items_rem) work items
  int split;                         // the counts above are 128-row blocks instead: a CTA's run may begin and end inside an item
  int n_tile, nnt, n_pad;      // output channels per pass, passes, nnt * n_tile
  int planes_all;              // chunk planes of the packed weights (all 64-channel planes and taps)
  int mb;                      // blocks per tile
  int lines_img;               // rbox * wbox: GEMM rows per image of a tile
  uint32_t inv_lines, inv_wbox; // ceil(2^20 / lines_img), ceil(2^20 / wbox)
  int a_stage_bytes, a_box_bytes, b_stage_bytes;
  int sa, sb, nacc, act;
  int b_resident;              // all weights stay in shared memory (one copy per CTA)
  int off_bias, off_stage, off_b, off_a, smem_bytes;
  int tmem_cols;
};

struct Shared {
  uint64_t a_full[kMaxA], a_empty[kMaxA];
  uint64_t b_full[kMaxB], b_empty[kMaxB];
  uint64_t b_all;              // resident weights have landed
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  uint32_t abort;
};

// 16-channel K steps of plane g
__device__ __forceinline__ int plane_steps(const RowsParams &p, int g) {
  const int left = p.c_in - 64 * g;
  return left >= 64 ? 4 : (left + 15) >> 4;
}

// work item -> (pass, image group, column strip, row tile); items are ordered (tile, pass)
struct Item {
  int nt, img0, xt, ty;
  __device__ __forceinline__ void of(const RowsParams &p, int item) {
    const int tile = item / p.nnt;
    nt = item - tile * p.nnt;
    const int strip = tile / p.tiles_y;
    ty = tile - strip * p.tiles_y;
    const int ig = strip / p.nxt;
    xt = strip - ig * p.nxt;
    img0 = ig * p.ni;
  }
};

// RESIDENT: all weights of the layer (a single output-channel pass, at most 128 KB) stay in shared memory:
// one copy per CTA instead of one stream per work item.  Compile-time, so that the streaming version's
// loops carry no switches.
template <bool RESIDENT>
__global__ void __launch_bounds__(kThreads, 1)
k_conv_tc_rows(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ RowsParams p,
               const void *__restrict__ w_packed, const float *__restrict__ bias,
               const __nv_bfloat16 *__restrict__ residual, __nv_bfloat16 *__restrict__ y, DcWsHeader *ws) {
  extern __shared__ __align__(1024) uint8_t smem_raw_base[];
  __shared__ __align__(8) Shared sh;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~uintptr_t(1023));
  uint8_t *smem_b = smem + p.off_b;
  uint8_t *smem_a = smem + p.off_a;              // 1024-byte aligned stages (the swizzle pattern repeats every 1024 bytes)
  uint8_t *smem_ones = smem + p.off_bias;        // 8 lines of the constant operand (1024-byte aligned)
  uint8_t *smem_bias = smem_ones + 1024;         // [n_pad][16 bytes]: bias as two bf16 terms, then n_tile zero rows

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile uint32_t *abort_flag = &sh.abort;

  const int bid = (int)blockIdx.x;
  // This CTA's run of work items.  When the plan balances by blocks (split), the run is counted in 128-row
  // blocks: its first item starts at block blk_first and its last one ends before blk_end; the tile and the
  // weights of such an item are still staged whole.
  int nitems = p.items_per + (bid < p.items_rem ? 1 : 0);
  int item0 = bid * p.items_per + (bid < p.items_rem ? bid : p.items_rem);
  int blk_first = 0, blk_end = p.mb;
  if (p.split) {
    const int u0 = item0, u1 = item0 + nitems - 1;           // first and last block of the run
    item0 = u0 / p.mb;
    const int item1 = u1 / p.mb;
    nitems = item1 - item0 + 1;
    blk_first = u0 - item0 * p.mb;
    blk_end = u1 - item1 * p.mb + 1;
  }

  {
    const int t = (int)threadIdx.x;
    bool did = false;
    if (t < p.sa) { mbar_init(&sh.a_full[t], 1); mbar_init(&sh.a_empty[t], kMmaWarps); did = true; }
    else if (t >= 32 && t < 32 + p.sb) { mbar_init(&sh.b_full[t - 32], 1); mbar_init(&sh.b_empty[t - 32], kMmaWarps); did = true; }
    else if (t >= 64 && t < 66) { mbar_init(&sh.acc_full[t - 64], kMmaWarps); mbar_init(&sh.acc_empty[t - 64], kEpiWarps); did = true; }
    else if (t == 96) { sh.abort = 0; mbar_init(&sh.b_all, 1); prefetch_tensormap(&map_a); did = true; }
    if (did) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  dc_pdl_enter();                                // nothing above touched global memory; everything below may
  __syncthreads();

  if (warp == 0) {
    // ================================================================== producer
    // The whole warp walks the loop (every lane observes the barriers itself); lane 0 announces the
    // bytes and issues the activation tile, the weight planes of a step are issued one per lane.
    {
      const uint32_t a_base0 = smem_u32(smem_a), b_base0 = smem_u32(smem_b);
      const char *wsrc = reinterpret_cast<const char *>(w_packed);
      int sa = 0, sb = 0;
      uint32_t pa = 0, pb = 0;
      bool ok = true;
      if (RESIDENT && lane == 0) {               // the whole packed buffer once
        const uint32_t all = (uint32_t)(p.planes_all * p.n_tile * 16);
        mbar_arrive_expect_tx(&sh.b_all, all);
        bulk_load(b_base0, wsrc, all, &sh.b_all);
      }
#pragma unroll 1
      for (int it = 0; it < nitems && ok; ++it) {
        Item q;
        q.of(p, item0 + it);
#pragma unroll 1
        for (int g = 0; g < p.planes && ok; ++g) {
          if (!warp_wait(&sh.a_empty[sa], pa ^ 1, abort_flag, ws, 0x10000u | sa)) { ok = false; break; }
          if (lane == 0) {
            // channels past c_in, pixels outside the image and images past the batch arrive as zeros
            mbar_arrive_expect_tx(&sh.a_full[sa], (uint32_t)p.a_box_bytes);
            tma_load_4d(a_base0 + (uint32_t)sa * (uint32_t)p.a_stage_bytes, &map_a, &sh.a_full[sa], 64 * g,
                        q.xt * p.tw - p.pad, q.ty * p.th - p.pad, q.img0);
          }
          if (++sa == p.sa) { sa = 0; pa ^= 1; }
          const int nsl = plane_steps(p, g);
          const int nplanes = p.k * nsl * 2;     // chunk planes of one (g, r) step
#pragma unroll 1
          for (int r = 0; r < p.k && !RESIDENT; ++r) {
            if (!warp_wait(&sh.b_empty[sb], pb ^ 1, abort_flag, ws, 0x20000u | sb)) { ok = false; break; }
            const uint32_t dst = b_base0 + (uint32_t)sb * (uint32_t)p.b_stage_bytes;
            const size_t plane0 = (size_t)g * p.k * p.k * 8 + (size_t)r * nplanes;
            if (lane == 0) mbar_arrive_expect_tx(&sh.b_full[sb], (uint32_t)(nplanes * p.n_tile * 16));
            __syncwarp();
            // the planes of a step are contiguous in the packed weights, with several passes too (there a
            // pass's rows of all planes are stored together): one bulk copy
            if (lane == 0)
              bulk_load(dst, wsrc + ((size_t)q.nt * p.planes_all + plane0) * p.n_tile * 16, (uint32_t)(nplanes * p.n_tile * 16),
                        &sh.b_full[sb]);
            if (++sb == p.sb) { sb = 0; pb ^= 1; }
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ---- consumer preparation
    if (warp == kMmaWarp) {
      tmem_alloc(&sh.tmem_base, (uint32_t)p.tmem_cols);
      tmem_relinquish();
    } else if (warp >= kFirstEpiWarp) {
      // The bias is added by the tensor core: one instruction per block multiplies a constant operand
      // (1.0 in the first two K elements of every line) with [bias as bf16, its bf16 remainder, 0, ...]
      // per output channel (exact to 16 mantissa bits) before the block's other instructions accumulate.
      // The constant operand is one 8-line group read sixteen times (group stride 0); with the 128-byte
      // swizzle the first 16-byte chunk of line r sits at chunk r.
      const int t0 = (int)threadIdx.x - kFirstEpiWarp * 32;
      for (int t = t0; t < 64; t += kEpiWarps * 32) {
        const int r = t >> 3, c = t & 7;
        reinterpret_cast<uint4 *>(smem_ones)[t] = make_uint4(c == r ? 0x3F803F80u : 0u, 0u, 0u, 0u);
      }
      for (int t = t0; t < p.n_pad + p.n_tile; t += kEpiWarps * 32) {
        uint32_t w0 = 0u;
        if (bias && t < p.c_out) {
          const float b = bias[t];
          const __nv_bfloat16 hi = __float2bfloat16_rn(b);
          const __nv_bfloat16 lo = __float2bfloat16_rn(b - __bfloat162float(hi));
          w0 = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16);
        }
        reinterpret_cast<uint4 *>(smem_bias)[t] = make_uint4(w0, 0u, 0u, 0u);
      }
      fence_proxy_async();                       // both are read by the tensor core (async proxy)
    }
    tc_fence_before();
    bar_sync(kBarConsumers, kConsumerThreads);
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp < kFirstEpiWarp) {
      // ================================================================== MMA issue
      const int mw = warp - kMmaWarp;
      // one election for the whole role: the warp stays converged and the same lane issues every instruction
      const bool leader = elect_one();
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_tile >> 3) << 17) | (8u << 24);
      const uint32_t b_hi = (128u >> 4) | (1u << 14);                 // no swizzle: 128 bytes between 8-row groups
      const uint32_t a_hi = (1024u >> 4) | (1u << 14) | (2u << 29);   // 128-byte swizzle: 1024 bytes between 8-row groups
      const uint32_t a_row0 = smem_u32(smem_a) >> 4, b_row0 = smem_u32(smem_b) >> 4;
      const uint32_t bias_row0 = smem_u32(smem_bias) >> 4, zero_row = bias_row0 + (uint32_t)p.n_pad;
      const uint64_t ones_desc = ((uint64_t)((1u << 14) | (2u << 29)) << 32) | (uint64_t)(((smem_u32(smem_ones) >> 4) & 0x3FFFu) | (1u << 16));
      int sa = 0, sb = 0;
      uint32_t pa = 0, pb = 0;
      uint32_t acc_ph[2] = {1u, 1u};             // parity this warp waits for on acc_empty (first use passes)
      bool ok = true;
      if (RESIDENT) {
        ok = warp_wait(&sh.b_all, 0, abort_flag, ws, 0x70000u);
        tc_fence_after();
      }
#pragma unroll 1
      for (int it = 0; it < nitems && ok; ++it) {
        const int set = p.nacc == 2 ? (it & 1) : 0;
        const int blk_lo = it == 0 ? blk_first : 0, blk_hi = it == nitems - 1 ? blk_end : p.mb;   // this run's blocks of the item
        if (!warp_wait(&sh.acc_empty[set], acc_ph[set], abort_flag, ws, 0x30000u | set)) break;
        acc_ph[set] ^= 1u;
        tc_fence_after();
        {
          // bias first (needs no load): it also initialises the accumulators of this warp's blocks
          Item iq;
          iq.of(p, item0 + it);
          const uint32_t bias_row = bias_row0 + (uint32_t)(iq.nt * p.n_tile);
          const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)((bias_row & 0x3FFFu) | ((zero_row - bias_row) << 16));
#pragma unroll 1
          for (int b = blk_lo + mw; b < blk_hi; b += kMmaWarps)
            if (leader) umma_bf16(tmem_base + (uint32_t)((set * p.mb + b) * p.n_tile), ones_desc, bd, idesc, 0u);
        }
#pragma unroll 1
        for (int g = 0; g < p.planes && ok; ++g) {
          if (!warp_wait(&sh.a_full[sa], pa, abort_flag, ws, 0x40000u | sa)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_stage = a_row0 + (uint32_t)sa * ((uint32_t)p.a_stage_bytes >> 4);
          const int nsl = plane_steps(p, g);
#pragma unroll 1
          for (int r = 0; r < p.k; ++r) {
            uint32_t b_stage;
            if (RESIDENT) {
              b_stage = b_row0 + (uint32_t)((g * p.k * p.k * 8 + r * p.k * nsl * 2) * p.n_tile);   // planes before this step
            } else {
              if (!warp_wait(&sh.b_full[sb], pb, abort_flag, ws, 0x50000u | sb)) { ok = false; break; }
              tc_fence_after();
              b_stage = b_row0 + (uint32_t)sb * ((uint32_t)p.b_stage_bytes >> 4);
            }
            // One lane issues the step's instructions in one stretch and the warp meets again behind it: with a
            // branch around every single instruction the warp diverged and met again each time, ~130 cycles per
            // instruction where the instruction itself takes ~50.  (Measured the same: every lane executing the
            // instruction under the leader's predicate, no branch at all.)
            if (leader) {
#pragma unroll 1
              for (int b = blk_lo + mw; b < blk_hi; b += kMmaWarps) {
                const uint32_t d = tmem_base + (uint32_t)((set * p.mb + b) * p.n_tile);
                // descriptors advance by adds only: +8 (one line) per tap column, +2 (32 bytes) per K step on
                // the activation side, two chunk planes per instruction on the weight side
                uint32_t a_lo = ((a_stage + (uint32_t)(b * 1024 + r * p.wbox * 8)) & 0x3FFFu) | (1u << 16);
                uint32_t b_lo = (b_stage & 0x3FFFu) | ((uint32_t)p.n_tile << 16);
                const uint32_t b_inc = 2u * (uint32_t)p.n_tile;
                if (nsl == 4) {                  // a full plane of 64 channels
#pragma unroll 1
                  for (int s = 0; s < p.k; ++s, a_lo += 8u) {
#pragma unroll
                    for (int sl = 0; sl < 4; ++sl) {
                      umma_bf16(d, ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + 2u * sl), ((uint64_t)b_hi << 32) | (uint64_t)b_lo, idesc, 1u);
                      b_lo += b_inc;
                    }
                  }
                } else {
#pragma unroll 1
                  for (int s = 0; s < p.k; ++s, a_lo += 8u) {
#pragma unroll 1
                    for (int sl = 0; sl < nsl; ++sl) {
                      umma_bf16(d, ((uint64_t)a_hi << 32) | (uint64_t)(a_lo + 2u * sl), ((uint64_t)b_hi << 32) | (uint64_t)b_lo, idesc, 1u);
                      b_lo += b_inc;
                    }
                  }
                }
              }
            }
            __syncwarp();
            if (!RESIDENT) {
              if (leader) umma_commit(&sh.b_empty[sb]);    // this warp is done with the weight stage
              if (++sb == p.sb) { sb = 0; pb ^= 1; }
            }
          }
          if (ok && leader) umma_commit(&sh.a_empty[sa]);  // ... and with the plane
          if (++sa == p.sa) { sa = 0; pa ^= 1; }
        }
        if (ok && leader) umma_commit(&sh.acc_full[set]);  // this warp's blocks of the item are complete
      }
    } else {
      // ================================================================== epilogue
      // Two warps per tensor-memory lane quadrant; blocks alternate between them.  A thread owns a
      // GEMM row = one pixel of the patch; valid ones store their n_tile channels 16 bytes at a time.
      const int ew = warp - kFirstEpiWarp;
      const int q = warp & 3, par = ew >> 2;
      const uint32_t tmem_row = tmem_base + ((uint32_t)(q * 32) << 16);
      // this warp's turn-around buffer, as 32-bit shared addresses: where this lane writes its pixel, and where it
      // reads the piece it stores of pixel lane / 4 (the three other pixels lie 8 * kStagePitch bytes apart)
      const uint32_t stage = smem_u32(smem + p.off_stage + ew * (32 * kStagePitch));
      // 16-byte piece g of pixel px sits at piece g ^ ((px >> 1) & 3) of the pixel's 64 bytes: the eight lanes of a
      // quarter warp then touch eight different 16-byte bank groups both when every lane writes piece g of its own
      // pixel and when four lanes read the four pieces of each of two neighbouring pixels
      const uint32_t stage_wr = stage + (uint32_t)lane * kStagePitch, swz_wr = (uint32_t)((lane >> 1) & 3);
      const uint32_t stage_rd = stage + (uint32_t)(lane >> 2) * kStagePitch +
                                (uint32_t)((lane & 3) ^ ((lane >> 3) & 3)) * 16u;
      uint32_t acc_ph[2] = {0u, 0u};
      const bool relu6 = p.act == DC_ACT_RELU6;
#pragma unroll 1
      for (int it = 0; it < nitems; ++it) {
        const int set = p.nacc == 2 ? (it & 1) : 0;
        Item iq;
        iq.of(p, item0 + it);
        if (!warp_wait(&sh.acc_full[set], acc_ph[set], abort_flag, ws, 0x60000u | set)) break;
        acc_ph[set] ^= 1u;
        tc_fence_after();
        const int x0 = iq.xt * p.tw, y0 = iq.ty * p.th;
        const int tw_valid = p.wo - x0 < p.tw ? p.wo - x0 : p.tw;
        const int th_valid = p.ho - y0 < p.th ? p.ho - y0 : p.th;
        const int ch0 = iq.nt * p.n_tile;
        const int nch = p.c_out - ch0 < p.n_tile ? p.c_out - ch0 : p.n_tile;   // multiple of 8
        const int blk_lo = it == 0 ? blk_first : 0, blk_hi = it == nitems - 1 ? blk_end : p.mb;   // this run's blocks of the item
#pragma unroll 1
        for (int b = blk_lo + par; b < blk_hi; b += 2) {
          const int pos = b * 128 + q * 32 + lane;
          // pos < 512 and the divisors are at most 256: multiplying by the rounded-up reciprocal is exact
          const int il = (int)(((uint32_t)pos * p.inv_lines) >> 20), rem = pos - il * p.lines_img;
          const int yy = (int)(((uint32_t)rem * p.inv_wbox) >> 20), xx = rem - yy * p.wbox;
          const bool valid = il < p.ni && iq.img0 + il < p.n_img && yy < th_valid && xx < tw_valid;
          // (the plan keeps the pixel count of the output below 2^31)
          const int pix = ((iq.img0 + il) * p.ho + (y0 + yy)) * p.wo + (x0 + xx);
          __nv_bfloat16 *dst = y + (size_t)pix * p.c_out + ch0;
          const __nv_bfloat16 *rp = residual ? residual + (size_t)pix * p.c_out + ch0 : nullptr;
          const uint32_t taddr = tmem_row + (uint32_t)((set * p.mb + b) * p.n_tile);
          // eight channels of this thread's pixel: skip input, activation -> eight bf16
          // (RELU and RES are compile-time: the per-pixel code carries no run-time switches)
          auto cook8 = [&](auto RELU, auto RES, const uint32_t *v, int ch) {
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[i]);     // the bias is in the accumulator already
            if (decltype(RES)::value && valid) {
              const uint4 rv = *reinterpret_cast<const uint4 *>(rp + ch);
              const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 rf = __bfloat1622float2(rb[i]);
                f[2 * i] += rf.x; f[2 * i + 1] += rf.y;
              }
            }
            uint4 ov;
            uint32_t *ow = reinterpret_cast<uint32_t *>(&ov);
            // ReLU6 on the rounded pairs: 0 and 6 are bf16 values and rounding is monotonic, so clamping in and
            // after the conversion gives the same values as clamping before it: the conversion clamps at zero
            // itself, one packed minimum against (6, 6) does the rest
#pragma unroll
            for (int i = 0; i < 4; ++i)
              ow[i] = decltype(RELU)::value ? min_bf16x2(pack_bf16x2_relu(f[2 * i], f[2 * i + 1]), 0x40C040C0u)
                                            : pack_bf16x2(f[2 * i], f[2 * i + 1]);
            return ov;
          };
          // 32 accumulator columns per read while they last.  A thread owns a pixel, so stored directly
          // its 16-byte pieces would land c_out * 2 bytes apart from its neighbours' (half-filled
          // sectors, 32 lines per instruction).  The warp instead turns the 32 pixels x 64 bytes around
          // in its staging buffer (64-byte pitch, pieces XOR-swizzled: conflict-free both ways) and writes them four lanes to a
          // pixel: every store instruction then fills eight whole 64-byte segments.
          const uint32_t vmask = __ballot_sync(0xffffffffu, valid);
          // the four pixels this lane helps to store (pixel i * 8 + lane / 4 of the warp's 32): their addresses
          // come from the lanes that own them, once per block
          uint8_t *px_ptr[4];                              // + 16 bytes per lane of the four that share a pixel
          bool px_on[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            px_ptr[i] = reinterpret_cast<uint8_t *>((uintptr_t)__shfl_sync(0xffffffffu, (unsigned long long)(uintptr_t)dst, i * 8 + (lane >> 2))) + (lane & 3) * 16;
            px_on[i] = (vmask >> (i * 8 + (lane >> 2))) & 1u;
          }
          auto emit32 = [&](auto RELU, auto RES, const uint32_t *v, int c0) {
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) sts_u4(stage_wr + (((uint32_t)g8 ^ swz_wr) << 4), cook8(RELU, RES, v + 8 * g8, c0 + 8 * g8));
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint4 piece = lds_u4(stage_rd + (uint32_t)(i * 8 * kStagePitch));
              if (px_on[i]) *reinterpret_cast<uint4 *>(px_ptr[i] + (size_t)c0 * 2) = piece;
            }
            __syncwarp();
          };
          auto channels = [&](auto RELU, auto RES) {
            int ch = 0;
#pragma unroll 1
            for (; ch + 32 <= nch; ch += 32) {
              uint32_t v[32];
              tmem_ld32(taddr + (uint32_t)ch, v);
              tmem_ld_wait();
              emit32(RELU, RES, v, ch);
            }
#pragma unroll 1
            for (; ch < nch; ch += 8) {
              uint32_t v[8];
              tmem_ld8(taddr + (uint32_t)ch, v);
              tmem_ld_wait();
              const uint4 ov = cook8(RELU, RES, v, ch);
              if (valid) *reinterpret_cast<uint4 *>(dst + ch) = ov;
            }
          };
          using T = std::true_type;
          using F = std::false_type;
          if (relu6) { if (rp) channels(T{}, T{}); else channels(T{}, F{}); }
          else { if (rp) channels(F{}, T{}); else channels(F{}, F{}); }
        }
        // this warp has read what it needs of the accumulator set
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.acc_empty[set]);
      }
    }
    // ---- consumer teardown
    if (*abort_flag) {
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    bar_sync(kBarConsumers, kConsumerThreads);
    if (warp == kMmaWarp) {
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

constexpr int kSmemBudget = 220 * 1024;
constexpr int kMaxLines = 128 * kMaxBlocks;      // GEMM rows of a tile
constexpr int kSlack = 1024;

bool rows_plan(int n, int h, int w, const dc_geom *g, int n_sm, RowsParams *p) {
  KOrder ko;
  dc_korder_init(&ko, g);
  if (!ko.rows) return false;
  const int ho = dc_out_extent(h, g->k, 1, g->pad), wo = dc_out_extent(w, g->k, 1, g->pad);
  if (ho <= 0 || wo <= 0) return false;
  if ((long long)n * h * w * g->c_in >= (1ll << 40) || (long long)n * ho * wo >= (1ll << 31)) return false;
  p->n_img = n; p->h = h; p->w = w; p->ho = ho; p->wo = wo;
  p->c_in = g->c_in; p->c_out = g->c_out;
  p->k = g->k; p->pad = g->pad;
  p->planes = dc_div_up(g->c_in, 64);
  p->n_tile = ko.n_tile; p->nnt = ko.nnt; p->n_pad = ko.n_pad;
  p->planes_all = ko.e_pad;
  // tile: as many rows as fit kMaxLines GEMM rows; whole small images several at a time.  Rows may be cut into
  // strips: of the first few strip counts that fit, the one with the fewest tiles per image wins (28 x 28 with a
  // 3 x 3 kernel: two strips of 14 columns x 14 rows make 4 tiles where full rows x 6 make 5)
  int nxt0 = 1;
  while (dc_div_up(wo, nxt0) + g->k - 1 > kMaxLines / g->k) ++nxt0;       // at least one output row per tile
  int th = 0, best_tiles = 0;
  p->nxt = 0;
  for (int cand = nxt0; cand <= nxt0 + 3 && cand <= wo; ++cand) {
    const int tw_c = dc_div_up(wo, cand), nxt_c = dc_div_up(wo, tw_c);
    int th_c = kMaxLines / (tw_c + g->k - 1) - (g->k - 1);
    if (th_c < 1) continue;
    if (th_c > ho) th_c = ho;
    const int tiles_c = nxt_c * dc_div_up(ho, th_c);
    if (p->nxt == 0 || tiles_c < best_tiles) { p->nxt = nxt_c; p->tw = tw_c; th = th_c; best_tiles = tiles_c; }
  }
  if (p->nxt == 0) return false;
  p->wbox = p->tw + g->k - 1;
  p->th = th;
  p->rbox = th + g->k - 1;
  p->lines_img = p->rbox * p->wbox;
  p->inv_lines = ((1u << 20) + (uint32_t)p->lines_img - 1) / (uint32_t)p->lines_img;
  p->inv_wbox = ((1u << 20) + (uint32_t)p->wbox - 1) / (uint32_t)p->wbox;
  p->ni = 1;
  if (th == ho && p->nxt == 1) {
    int ni_max = kMaxLines / p->lines_img;
    if (ni_max > n) ni_max = n;
    if (ni_max > 8) ni_max = 8;
    if (ni_max < 1) ni_max = 1;
    // Fewer images per tile where that fills the machine: a work item takes in its activation planes and its
    // pass's weights from L2, and the launch lasts as long as the CTA with the most items.  Cost of a choice =
    // items per CTA x (bytes of an item + 64 KB for the item's own chain of waits); a smaller count must win
    // by a tenth.  960 -> 160, 1 x 1, 128 images of 7 x 7: two images per tile (128 items) instead of five (52).
    const long long w_item = (long long)ko.e_pad * p->n_tile * 16;
    long long best_cost = 0;
    p->ni = ni_max;
    for (int c = ni_max; c >= 1; --c) {
      const long long items_c = (long long)dc_div_up(n, c) * p->nnt;
      const long long per_cta = (items_c + n_sm - 1) / n_sm;
      const long long cost = per_cta * ((long long)c * p->lines_img * 128 * p->planes + w_item + 64 * 1024);
      if (c == ni_max || cost * 10 < best_cost * 9) { best_cost = cost; p->ni = c; }
    }
  }
  if (p->wbox > 256 || p->rbox > 256) return false;
  p->tiles_y = dc_div_up(ho, th);
  p->img_groups = dc_div_up(n, p->ni);
  const int last = (p->ni - 1) * p->lines_img + (th - 1) * p->wbox + p->tw;    // GEMM rows up to the last valid one
  p->mb = dc_div_up(last, 128);
  if (p->mb > kMaxBlocks) return false;
  p->nacc = (2 * p->mb * p->n_tile <= 512) ? 2 : 1;
  if (p->nacc * p->mb * p->n_tile > 512) return false;
  int cols = 32;
  while (cols < p->nacc * p->mb * p->n_tile) cols *= 2;
  p->tmem_cols = cols;
  const long long items = (long long)p->img_groups * p->nxt * p->tiles_y * p->nnt;
  if (items >= (1ll << 30)) return false;
  p->grid = items < n_sm ? (int)items : n_sm;
  p->items_per = (int)(items / p->grid);
  p->items_rem = (int)(items % p->grid);
  // Where whole items leave some CTAs a block more than an even split would (160 -> 960, 3 x 3 at 7 x 7: 344
  // items of two blocks on 148 SMs, three items = six blocks on 48 of them against five by blocks), the runs are
  // cut by blocks: an item at a run's end is then shared by two CTAs, each staging its tile and weights.
  p->split = 0;
  if (p->mb > 1) {
    const long long units = items * p->mb;
    const int grid_u = units < n_sm ? (int)units : n_sm;
    const long long whole = (items / p->grid + (items % p->grid ? 1 : 0)) * p->mb, cut = units / grid_u + (units % grid_u ? 1 : 0);
    if (cut * 8 <= whole * 7 && units < (1ll << 30)) {     // worth it from an eighth less (a shared item is staged twice)
      p->split = 1;
      p->grid = grid_u;
      p->items_per = (int)(units / grid_u);
      p->items_rem = (int)(units % grid_u);
    }
  }
  p->a_box_bytes = p->ni * p->lines_img * 128;
  p->a_stage_bytes = (int)dc_round_up((size_t)p->a_box_bytes, 1024);
  p->b_stage_bytes = (int)dc_round_up((size_t)g->k * 4 * 2 * p->n_tile * 16, 1024);
  // Layout: bias, activation stages, weight stages.  A block's 128 GEMM rows plus the tap shift may
  // reach up to ~200 lines (25 KB) past its stage; behind the last activation stage that lands in
  // the weight stages, which are larger (what is read there only feeds rows that are dropped).
  p->off_bias = 0;
  p->off_stage = (int)dc_round_up((size_t)1024 + (size_t)(p->n_pad + p->n_tile) * 16, 128);   // constant operand, bias rows, zero rows
  p->off_a = (int)dc_round_up((size_t)p->off_stage + kEpiWarps * 32 * kStagePitch, 1024);
  // rings: weights first (they are the larger stream), then activation planes
  int sa = 2, sb = 2;
  // Small weights of a single pass stay resident where a work item would otherwise stream more weight than
  // activation bytes (many input planes, or a k x k kernel on few): then it streams its activation planes only.
  // (For 1 x 1 layers of one or two planes the weight stream is small beside the activations and the resident
  // version measured no faster.)
  const long long b_all = (long long)dc_round_up((size_t)ko.e_pad * p->n_tile * 16, 1024);
  p->b_resident = (p->nnt == 1 && b_all <= 128 * 1024 && (p->planes >= 3 || b_all >= 2ll * p->a_stage_bytes)) ? 1 : 0;
  auto total = [&](int a, int b) {
    const long long wbytes = p->b_resident ? b_all : (long long)b * p->b_stage_bytes;
    const long long tail = wbytes >= 26 * 1024 ? kSlack : 26 * 1024 - wbytes + kSlack;   // room for the overrun
    return 1024ll + p->off_a + wbytes + (long long)a * p->a_stage_bytes + tail;
  };
  if (p->b_resident && total(sa, sb) > kSmemBudget) p->b_resident = 0;
  if (total(sa, sb) > kSmemBudget) return false;
  while (!p->b_resident && sb < kFirstB && total(sa, sb + 1) <= kSmemBudget) ++sb;
  while (sa < kFirstA && total(sa + 1, sb) <= kSmemBudget) ++sa;
  // Layers of many input planes with small stages (deep 1 x 1 layers: 10-30 KB per step) are bound by the
  // bytes in flight (a stage comes back ~1 us after it was asked for), so what shared memory is left deepens
  // both rings in turn.
  for (bool grew = true; grew;) {
    grew = false;
    if (!p->b_resident && sb < kMaxB && total(sa, sb + 1) <= kSmemBudget) { ++sb; grew = true; }
    if (sa < kMaxA && total(sa + 1, sb) <= kSmemBudget) { ++sa; grew = true; }
  }
  p->sa = sa; p->sb = sb;
  p->off_b = p->off_a + sa * p->a_stage_bytes;
  p->smem_bytes = (int)total(sa, sb);
  return true;
}

}  // namespace

bool dc_conv_rows_supported(int n, int h, int w, const dc_geom *g) {
  RowsParams p;
  return rows_plan(n, h, w, g, dc_sm_count(), &p);
}

dc_status dc_launch_conv_rows(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                              const float *bias, dc_act act, const void *residual, void *y, void *workspace,
                              cudaStream_t stream) {
  RowsParams p;
  const int n_sm = dc_sm_count();
  if (!rows_plan(n, h, w, g, n_sm, &p)) return DC_ERR_UNSUPPORTED;
  p.act = (int)act;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return DC_ERR_CUDA;
  CUtensorMap map_a;
  {
    const cuuint64_t C = (cuuint64_t)g->c_in;
    cuuint64_t gdim[4] = {C, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    cuuint64_t gstr[3] = {2 * C, (cuuint64_t)w * C * 2, (cuuint64_t)h * w * C * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)p.wbox, (cuuint32_t)p.rbox, (cuuint32_t)p.ni};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(x), gdim, gstr, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DC_ERR_CUDA;
  }
  static unsigned char attr_done[kDcMaxDevices];
  static unsigned char attr_done_r[kDcMaxDevices];
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_tc_rows<false>, kSmemBudget, attr_done));
  DC_CUDA_OK(dc_set_max_smem_once(k_conv_tc_rows<true>, kSmemBudget, attr_done_r));
  const cudaError_t le = dc_launch_pdl(p.b_resident ? k_conv_tc_rows<true> : k_conv_tc_rows<false>, dim3(p.grid), dim3(kThreads), (size_t)p.smem_bytes, stream, map_a, p,
                                       w_packed, bias, (const __nv_bfloat16 *)residual, (__nv_bfloat16 *)y,
                                       (DcWsHeader *)workspace);
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
