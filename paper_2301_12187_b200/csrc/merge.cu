// BN folding, composition of a run of convolutions into one convolution, and weight repacking.
// fp32 FMA arithmetic on CUDA cores: the merged weights must match an fp64 evaluation of the
// same formula to 1e-5 relative, which rules out reduced-precision tensor-core math.
#include <vector>

#include "common.cuh"

// ----------------------------------------------------------------------------------------------
// kernels
// ----------------------------------------------------------------------------------------------

#define DC_FOLD_MAX 16
struct FoldTable {
  const float *w[DC_FOLD_MAX], *b[DC_FOLD_MAX], *gamma[DC_FOLD_MAX], *beta[DC_FOLD_MAX],
      *mean[DC_FOLD_MAX], *var[DC_FOLD_MAX];
  float *w_out[DC_FOLD_MAX], *b_out[DC_FOLD_MAX];
  float eps[DC_FOLD_MAX];
  int c_out[DC_FOLD_MAX], per_out[DC_FOLD_MAX];
  int n;
};

// blockIdx.y = layer; grid-stride over that layer's weights.  g = gamma / sqrt(var + eps).
__global__ void k_fold_bn(const __grid_constant__ FoldTable t) {
  const int l = blockIdx.y;
  const int per = t.per_out[l];
  const int total = t.c_out[l] * per;
  const bool has_bn = t.gamma[l] != nullptr;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int o = i / per;
    float g = 1.f;
    if (has_bn) g = t.gamma[l][o] / sqrtf(t.var[l][o] + t.eps[l]);
    t.w_out[l][i] = g * t.w[l][i];
    if (i - o * per == 0) {
      float b = t.b[l] ? t.b[l][o] : 0.f;
      t.b_out[l][o] = has_bn ? fmaf(b - t.mean[l][o], g, t.beta[l][o]) : b;
    }
  }
}

// One piece of a run while it is being merged: a dense kernel [c_out][c_in][k][k] or a diagonal
// (depthwise) one [c][k][k], with its bias and accumulated stride.
struct Piece {
  const float *w;
  const float *b;
  int c_in, c_out, k, stride, diag;
  int ident;   // 1: the piece stands for w + I (identity kernel of a skip addition: +1 on the centre
               // tap of every (c, c) pair), added where the weights are read instead of by a launch
};

__device__ __forceinline__ float piece_dense_at(const Piece &p, int o, int i, int u, int v) {
  float w = p.w[(((size_t)o * p.c_in + i) * p.k + u) * p.k + v];
  const int ctr = (p.k - 1) / 2;
  if (p.ident && o == i && u == ctr && v == ctr) w += 1.f;
  return w;
}
__device__ __forceinline__ float piece_diag_at(const Piece &p, int c, int u, int v) {
  float w = p.w[((size_t)c * p.k + u) * p.k + v];
  const int ctr = (p.k - 1) / 2;
  if (p.ident && u == ctr && v == ctr) w += 1.f;
  return w;
}

// b'[o] = b2[o] + sum_c (sum_taps W2[o,c]) * b1[c]; one warp per output channel.  Runs in the
// tail blocks of the composition kernels (block index `blk` counted from the first bias block).
__device__ __forceinline__ void compose_bias_block(const Piece &first, const Piece &second, float *out, int blk) {
  const int warp = (blk * (int)blockDim.x + (int)threadIdx.x) / 32, lane = threadIdx.x % 32;
  if (warp >= second.c_out) return;
  const int o = warp, t2 = second.k * second.k;
  float acc = 0.f;
  if (second.diag) {
    if (lane == 0) {
      float ws = second.ident ? 1.f : 0.f;
      for (int t = 0; t < t2; ++t) ws += second.w[(size_t)o * t2 + t];
      acc = ws * first.b[o];
    }
  } else {
    for (int c = lane; c < second.c_in; c += 32) {
      float ws = (second.ident && c == o) ? 1.f : 0.f;
      for (int t = 0; t < t2; ++t) ws += second.w[((size_t)o * second.c_in + c) * t2 + t];
      acc = fmaf(ws, first.b[c], acc);
    }
  }
  for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
  if (lane == 0) out[o] = second.b[o] + acc;
}
static int bias_blocks(int c_out, int threads) { return dc_div_up(c_out * 32, threads); }

// dense (second) o dense (first) for large results:  out[o][j] = sum_r A[o][r] * B[r][j] with
//   r = (c, u2, v2),  j = (i, u', v'),  A = W2 as stored,
//   B[r][j] = W1[c][i][u' - s1*u2][v' - s1*v2]  (0 when the tap falls outside W1):
// a gathered-operand SGEMM with register-staged double buffering.  Tile (16 * TM) x 64 outputs, 256 threads, TM x 4 outputs per thread, reduction slices of
// 16 rows: while a slice is multiplied from shared memory the next one's operands are already on
// their way into registers, so the loads' round trips to L2 hide behind the arithmetic instead of
// alternating with it.  Same reduction order (c, u2, v2) as the other composition kernels.
constexpr int kDtK = 16;                         // reduction rows per slice
template <int TM>
__global__ void __launch_bounds__(256) k_compose_dd_tiled(Piece first, Piece second, float *out, float *b_out,
                                                          int kk, int gx, int gy) {
  constexpr int BM = 16 * TM, PA = BM + 4, PB = 64 + 4;
  __shared__ __align__(16) float As[2][kDtK][PA];
  __shared__ __align__(16) float Bs[2][kDtK][PB];
  if ((int)blockIdx.x >= gx * gy) {
    compose_bias_block(first, second, b_out, (int)blockIdx.x - gx * gy);
    return;
  }
  const int ctr1 = (first.k - 1) / 2, ctr2 = (second.k - 1) / 2;
  const int k1 = first.k, k2 = second.k, s1 = first.stride, t2sz = k2 * k2;
  const int c0 = first.c_in, c1 = first.c_out, c2 = second.c_out;
  const int R = c1 * t2sz, J = c0 * kk * kk;
  const int o0 = ((int)blockIdx.x / gx) * BM, j0 = ((int)blockIdx.x % gx) * 64;
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
  // loads: A element (o = o0 + (t >> 4) + 16 q, r = t & 15), B element (r = (t >> 6) + 4 u, j = j0 + (t & 63))
  const int ar = t & 15, ao = t >> 4;
  const int jj = t & 63, j = j0 + jj, br = t >> 6;
  const int bi = j / (kk * kk), btp = j - bi * kk * kk, bup = btp / kk, bvp = btp - bup * kk;
  // fetch() only issues the loads (from a safe address where the element is structurally zero) and keeps what
  // decides the element's value as two bit masks; the values are first touched in stage(), behind the
  // arithmetic on the current slice, so the loads' round trips hide behind it.  (With the selects in fetch()
  // every warp waited for its loads before it started on the slice.)
  float av[TM], bv[4];
  uint32_t a_ok, a_id, b_ok, b_id;
  auto fetch = [&](int r0) {
    const int ra = r0 + ar;
    a_ok = a_id = b_ok = b_id = 0u;
#pragma unroll
    for (int q = 0; q < TM; ++q) {
      const int o = o0 + ao + 16 * q;
      const bool ok = o < c2 && ra < R;
      av[q] = second.w[ok ? (size_t)o * R + ra : 0];
      a_ok |= (ok ? 1u : 0u) << q;
      a_id |= ((ok && second.ident && ra == (o * k2 + ctr2) * k2 + ctr2) ? 1u : 0u) << q;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = r0 + br + 4 * u;
      int c = r, u2 = 0, v2 = 0;
      if (t2sz != 1) {
        c = r / t2sz;
        const int t2 = r - c * t2sz;
        u2 = t2 / k2;
        v2 = t2 - u2 * k2;
      }
      const int u1 = bup - s1 * u2, v1 = bvp - s1 * v2;
      const bool ok = r < R && j < J && u1 >= 0 && u1 < k1 && v1 >= 0 && v1 < k1;
      bv[u] = first.w[ok ? (((size_t)c * c0 + bi) * k1 + u1) * k1 + v1 : 0];
      b_ok |= (ok ? 1u : 0u) << u;
      b_id |= ((ok && first.ident && c == bi && u1 == ctr1 && v1 == ctr1) ? 1u : 0u) << u;
    }
  };
  auto stage = [&](int buf) {
#pragma unroll
    for (int q = 0; q < TM; ++q)
      As[buf][ar][ao + 16 * q] = ((a_ok >> q) & 1u) ? (((a_id >> q) & 1u) ? av[q] + 1.f : av[q]) : 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      Bs[buf][br + 4 * u][jj] = ((b_ok >> u) & 1u) ? (((b_id >> u) & 1u) ? bv[u] + 1.f : bv[u]) : 0.f;
  };
  float acc[TM][4] = {};
  fetch(0);
  stage(0);
  __syncthreads();
  int buf = 0;
  for (int r0 = 0; r0 < R; r0 += kDtK) {
    const bool more = r0 + kDtK < R;
    if (more) fetch(r0 + kDtK);
#pragma unroll
    for (int rr = 0; rr < kDtK; ++rr) {
      float a[TM];
#pragma unroll
      for (int q = 0; q < TM; q += 4) {
        const float4 a4 = *reinterpret_cast<const float4 *>(&As[buf][rr][ty * TM + q]);
        a[q] = a4.x; a[q + 1] = a4.y; a[q + 2] = a4.z; a[q + 3] = a4.w;
      }
      const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[buf][rr][tx * 4]);
      const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int p = 0; p < TM; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(a[p], b[q], acc[p][q]);
    }
    if (more) stage(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
#pragma unroll
  for (int p = 0; p < TM; ++p) {
    const int o = o0 + ty * TM + p;
    if (o >= c2) continue;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int jo = j0 + tx * 4 + q;
      if (jo < J) out[(size_t)o * J + jo] = acc[p][q];
    }
  }
}

// dense 3x3 (stride 1) followed by dense 3x3, large channel counts (VGG-style runs): the result's
// 5x5 kernel of one (o, i) pair is the sum over c of the full 2-D product of W2[o][c] (3x3) and
// W1[c][i] (3x3), 81 multiply-adds per c, none of them with a structural zero -- the gathered GEMM
// of the kernels above multiplies all 9 x 25 (tap, position) pairs, 64 % of which are zero.
// CTA: 16 output channels x 32 input channels, 256 threads, a thread owns one o and two i (50
// accumulators); slices of 8 intermediate channels are staged in shared memory with the next slice's
// loads in flight (taps padded to 12 floats, read as three 16-byte vectors).  blockIdx.x walks the
// tiles (i fastest); the blocks after them compute the bias.
// At most 128 registers per thread, so that two CTAs share an SM and one's loads hide behind the other's
// arithmetic (c = 512: 1.31 -> 0.97 ms).  Tiles of 8 output channels in CTAs of 128 threads, for results with
// fewer tiles than two per SM, were measured and spill (c = 256: 209 -> 302 us): not kept.
constexpr int kPolyC = 8;
__global__ void __launch_bounds__(256, 2) k_compose_poly33(Piece first, Piece second, float *out, float *b_out, int gx, int gy) {
  __shared__ __align__(16) float W2s[2][16][kPolyC][12];   // [o][c][tap]
  __shared__ __align__(16) float W1s[2][kPolyC][32][12];   // [c][i][tap]
  if ((int)blockIdx.x >= gx * gy) {
    compose_bias_block(first, second, b_out, (int)blockIdx.x - gx * gy);
    return;
  }
  const int c0 = first.c_in, c1 = first.c_out, c2 = second.c_out;
  const int o0 = ((int)blockIdx.x / gx) * 16, i0 = ((int)blockIdx.x % gx) * 32;
  const int t = threadIdx.x, ol = t >> 4, il = t & 15;       // this thread's o, and i = il, il + 16
  // loads of a slice: W2: 16 o x 8 c x 9 = 1152 floats, W1: 8 c x 32 i x 9 = 2304 floats
  constexpr int N2 = (16 * kPolyC * 9 + 255) / 256, N1 = (kPolyC * 32 * 9) / 256;
  // fetch() only issues the loads and notes in bit masks what decides each element's value; the values are
  // first touched in stage(), behind the arithmetic on the current slice (see k_compose_dd_tiled).
  float r2[N2], r1[N1];
  uint32_t ok2, id2, ok1, id1;
  auto fetch = [&](int cs) {
    ok2 = id2 = ok1 = id1 = 0u;
#pragma unroll
    for (int q = 0; q < N2; ++q) {
      const int e = t + 256 * q;                 // (o, c, tap): taps of one (o, c) are contiguous in memory
      const int tap = e % 9, oc = e / 9, cl = oc % kPolyC, o = o0 + oc / kPolyC, c = cs + cl;
      const bool ok = e < 16 * kPolyC * 9 && o < c2 && c < c1;
      r2[q] = second.w[ok ? ((size_t)o * c1 + c) * 9 + tap : 0];
      ok2 |= (ok ? 1u : 0u) << q;
      id2 |= ((ok && second.ident && o == c && tap == 4) ? 1u : 0u) << q;
    }
#pragma unroll
    for (int q = 0; q < N1; ++q) {
      const int e = t + 256 * q;                 // (c, i, tap)
      const int tap = e % 9, ci = e / 9, i = i0 + ci % 32, c = cs + ci / 32;
      const bool ok = c < c1 && i < c0;
      r1[q] = first.w[ok ? ((size_t)c * c0 + i) * 9 + tap : 0];
      ok1 |= (ok ? 1u : 0u) << q;
      id1 |= ((ok && first.ident && c == i && tap == 4) ? 1u : 0u) << q;
    }
  };
  auto stage = [&](int buf) {
#pragma unroll
    for (int q = 0; q < N2; ++q) {
      const int e = t + 256 * q, tap = e % 9, oc = e / 9;
      if (e < 16 * kPolyC * 9)
        W2s[buf][oc / kPolyC][oc % kPolyC][tap] = ((ok2 >> q) & 1u) ? (((id2 >> q) & 1u) ? r2[q] + 1.f : r2[q]) : 0.f;
    }
#pragma unroll
    for (int q = 0; q < N1; ++q) {
      const int e = t + 256 * q, tap = e % 9, ci = e / 9;
      W1s[buf][ci / 32][ci % 32][tap] = ((ok1 >> q) & 1u) ? (((id1 >> q) & 1u) ? r1[q] + 1.f : r1[q]) : 0.f;
    }
  };
  float acc[2][25] = {};
  fetch(0);
  stage(0);
  __syncthreads();
  int buf = 0;
  for (int cs = 0; cs < c1; cs += kPolyC) {
    const bool more = cs + kPolyC < c1;
    if (more) fetch(cs + kPolyC);
#pragma unroll 4
    for (int cl = 0; cl < kPolyC; ++cl) {
      float a[12], b[2][12];
#pragma unroll
      for (int v = 0; v < 3; ++v) {
        *reinterpret_cast<float4 *>(a + 4 * v) = *reinterpret_cast<const float4 *>(&W2s[buf][ol][cl][4 * v]);
        *reinterpret_cast<float4 *>(b[0] + 4 * v) = *reinterpret_cast<const float4 *>(&W1s[buf][cl][il][4 * v]);
        *reinterpret_cast<float4 *>(b[1] + 4 * v) = *reinterpret_cast<const float4 *>(&W1s[buf][cl][il + 16][4 * v]);
      }
#pragma unroll
      for (int u2 = 0; u2 < 3; ++u2)
#pragma unroll
        for (int v2 = 0; v2 < 3; ++v2)
#pragma unroll
          for (int u1 = 0; u1 < 3; ++u1)
#pragma unroll
            for (int v1 = 0; v1 < 3; ++v1) {
              acc[0][(u1 + u2) * 5 + v1 + v2] = fmaf(a[u2 * 3 + v2], b[0][u1 * 3 + v1], acc[0][(u1 + u2) * 5 + v1 + v2]);
              acc[1][(u1 + u2) * 5 + v1 + v2] = fmaf(a[u2 * 3 + v2], b[1][u1 * 3 + v1], acc[1][(u1 + u2) * 5 + v1 + v2]);
            }
    }
    if (more) stage(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
  const int o = o0 + ol;
  if (o < c2) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int i = i0 + il + 16 * h;
      if (i < c0) {
        float *dst = out + ((size_t)o * c0 + i) * 25;
#pragma unroll
        for (int e = 0; e < 25; ++e) dst[e] = acc[h][e];
      }
    }
  }
}

// dense o dense for small results (the usual case: a merged kernel has a few thousand elements):
// 8 x 32 output tile, one output per thread, so that even a 24 x 216 result spreads over 21 CTAs;
// operands staged in shared memory a slice of up to kDdSmallSlice reduction rows at a time, all of
// a slice's loads in flight together.  Same reduction order (c, u2, v2) as the large-tile kernel.
// Blocks [0, gx*gy) are the tiles (x fastest); the blocks after them compute the bias.
constexpr int kDdSmallSlice = 256;
__global__ void __launch_bounds__(256) k_compose_dd_small(Piece first, Piece second, float *out, float *b_out,
                                                          int kk, int gx, int gy) {
  __shared__ float As[kDdSmallSlice][8];
  __shared__ float Bs[kDdSmallSlice][32];
  __shared__ unsigned char tap_u[64], tap_v[64];     // (u2, v2) of tap t2 of the second kernel
  if ((int)blockIdx.x >= gx * gy) {
    compose_bias_block(first, second, b_out, (int)blockIdx.x - gx * gy);
    return;
  }
  const int ctr1 = (first.k - 1) / 2, ctr2 = (second.k - 1) / 2;
  const int k1 = first.k, k2 = second.k, s1 = first.stride, t2sz = k2 * k2;
  const int c0 = first.c_in, c1 = first.c_out, c2 = second.c_out;
  const int R = c1 * t2sz, J = c0 * kk * kk;
  const int o0 = ((int)blockIdx.x / gx) * 8, j0 = ((int)blockIdx.x % gx) * 32;
  const int t = threadIdx.x, ol = t >> 5, jl = t & 31;
  if (t < t2sz) { tap_u[t] = (unsigned char)(t / k2); tap_v[t] = (unsigned char)(t % k2); }
  __syncthreads();
  const int j = j0 + jl, o = o0 + ol;
  const int bi = j / (kk * kk), btp = j - bi * kk * kk, bup = btp / kk, bvp = btp - bup * kk;
  float acc = 0.f;
  for (int r0 = 0; r0 < R; r0 += kDdSmallSlice) {
    const int rows = R - r0 < kDdSmallSlice ? R - r0 : kDdSmallSlice;
    // Operand loads go out in batches with no branch between them (an element outside the operand
    // reads element 0 and is zeroed afterwards: a load behind a branch waits for the one before it).
    // A[o][r]: a warp reads 32 consecutive r of one output channel
    {
      float av[kDdSmallSlice / 32];
#pragma unroll
      for (int u = 0; u < kDdSmallSlice / 32; ++u) {
        const int rr = jl + 32 * u, r = r0 + (rr < rows ? rr : rows - 1);
        const bool ok = o < c2 && rr < rows;
        const float x = second.w[ok ? (size_t)o * R + r : 0];
        av[u] = ok ? ((second.ident && r == (o * k2 + ctr2) * k2 + ctr2) ? x + 1.f : x) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < kDdSmallSlice / 32; ++u)
        if (jl + 32 * u < rows) As[jl + 32 * u][ol] = av[u];
    }
    // B[r][j]: a warp reads one row r, 32 consecutive j
    for (int rb = ol; rb < rows; rb += 64) {
      float bv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int rr = rb + 8 * u, r = r0 + (rr < rows ? rr : rows - 1);
        int c = r, t2 = 0;
        if (t2sz != 1) { c = r / t2sz; t2 = r - c * t2sz; }
        const int u1 = bup - s1 * tap_u[t2], v1 = bvp - s1 * tap_v[t2];
        const bool ok = j < J && u1 >= 0 && u1 < k1 && v1 >= 0 && v1 < k1;
        const float x = first.w[ok ? (((size_t)c * c0 + bi) * k1 + u1) * k1 + v1 : 0];
        bv[u] = ok ? ((first.ident && c == bi && u1 == ctr1 && v1 == ctr1) ? x + 1.f : x) : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (rb + 8 * u < rows) Bs[rb + 8 * u][jl] = bv[u];
    }
    __syncthreads();
#pragma unroll 8
    for (int rr = 0; rr < rows; ++rr) acc = fmaf(As[rr][ol], Bs[rr][jl], acc);
    __syncthreads();
  }
  if (o < c2 && j < J) out[(size_t)o * J + j] = acc;
}

// dense k x k (second) after a dense 1x1 with stride 1 (first): every tap sum has one term,
//   out[o][i][t] = sum_c W2[o][c][t] * W1[c][i],
// so the general gather would multiply k*k - 1 zeros per product.  blockIdx.y = o; the CTA stages
// W2[o] ([c1][k*k], at most kAfter1x1MaxFloats) in shared memory, a thread owns one (i, t) and
// walks c.  Blocks with blockIdx.y == c_out compute the bias.
constexpr int kAfter1x1MaxFloats = 11264;
__global__ void __launch_bounds__(256) k_compose_after_1x1(Piece first, Piece second, float *out, float *b_out) {
  __shared__ float Ws[kAfter1x1MaxFloats];
  const int c0 = first.c_in, c1 = first.c_out, c2 = second.c_out, kk = second.k * second.k, J = c0 * kk;
  if ((int)blockIdx.y >= c2) {
    compose_bias_block(first, second, b_out, (int)blockIdx.x);
    return;
  }
  const int o = blockIdx.y, ctr = ((second.k - 1) / 2) * (second.k + 1);
  for (int e = threadIdx.x; e < c1 * kk; e += blockDim.x) {
    float w = second.w[(size_t)o * c1 * kk + e];
    if (second.ident && e == o * kk + ctr) w += 1.f;
    Ws[e] = w;
  }
  __syncthreads();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= J) return;
  const int i = j / kk, t = j - i * kk;
  const float *w1 = first.w + i, *w2 = Ws + t;
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  int c = 0;
  for (; c + 4 <= c1; c += 4) {
    const float b0 = w1[(size_t)(c + 0) * c0], b1 = w1[(size_t)(c + 1) * c0];
    const float b2 = w1[(size_t)(c + 2) * c0], b3 = w1[(size_t)(c + 3) * c0];
    acc0 = fmaf(w2[(c + 0) * kk], b0, acc0);
    acc1 = fmaf(w2[(c + 1) * kk], b1, acc1);
    acc2 = fmaf(w2[(c + 2) * kk], b2, acc2);
    acc3 = fmaf(w2[(c + 3) * kk], b3, acc3);
  }
  for (; c < c1; ++c) acc0 = fmaf(w2[c * kk], w1[(size_t)c * c0], acc0);
  float acc = (acc0 + acc1) + (acc2 + acc3);
  if (first.ident && i < c1) acc += w2[i * kk];      // first + I: the c == i term once more
  out[(size_t)o * J + j] = acc;
}

// Compositions in which at least one operand is diagonal: one thread per output element.
//   second diag, first dense: out[o,i,u',v'] = sum_{u2,v2} W2[o,u2,v2] * W1[o,i,u1,v1]
//   second dense, first diag: out[o,i,u',v'] = sum_{u2,v2} W2[o,i,u2,v2] * W1[i,u1,v1]
//   both diag:                out[c,u',v']   = sum_{u2,v2} W2[c,u2,v2]   * W1[c,u1,v1]
// Blocks [0, nb) walk the elements; the blocks after them compute the bias.
// Depthwise K2 x K2 after a dense 1x1 with stride 1 (expand -> depthwise): the tap sums have one
// term, out[o][i][t] = W2[o][t] * W1[o][i].
template <int K2>
__device__ __forceinline__ void compose_diag_after_1x1(const Piece &first, const Piece &second, float *out, int total,
                                                       int nb) {
  constexpr int KK = K2 * K2, CTR = (K2 / 2) * (K2 + 1);
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += nb * blockDim.x) {
    const int t = idx % KK, rest = idx / KK;
    const int o = rest / first.c_in, i = rest - o * first.c_in;
    float w2 = second.w[(size_t)o * KK + t];
    if (second.ident && t == CTR) w2 += 1.f;
    float w1 = first.w[rest];
    if (first.ident && o == i) w1 += 1.f;
    out[idx] = fmaf(w2, w1, 0.f);
  }
}

__global__ void k_compose_diag(Piece first, Piece second, float *out, float *b_out, int kk, int total, int nb) {
  if ((int)blockIdx.x >= nb) {
    compose_bias_block(first, second, b_out, (int)blockIdx.x - nb);
    return;
  }
  if (second.diag && !first.diag && first.k == 1 && first.stride == 1) {
    if (second.k == 3) { compose_diag_after_1x1<3>(first, second, out, total, nb); return; }
    if (second.k == 5) { compose_diag_after_1x1<5>(first, second, out, total, nb); return; }
  }
  const int k1 = first.k, k2 = second.k, s1 = first.stride;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += nb * blockDim.x) {
    int vp = idx % kk, up = (idx / kk) % kk, rest = idx / (kk * kk);
    int o, i;
    if (first.diag && second.diag) { o = rest; i = rest; }
    else { i = rest % first.c_in; o = rest / first.c_in; }
    float acc = 0.f;
    for (int u2 = 0; u2 < k2; ++u2) {
      int u1 = up - s1 * u2;
      if (u1 < 0 || u1 >= k1) continue;
      for (int v2 = 0; v2 < k2; ++v2) {
        int v1 = vp - s1 * v2;
        if (v1 < 0 || v1 >= k1) continue;
        float w2 = second.diag ? piece_diag_at(second, o, u2, v2) : piece_dense_at(second, o, i, u2, v2);
        float w1 = first.diag ? piece_diag_at(first, i, u1, v1) : piece_dense_at(first, o, i, u1, v1);
        acc = fmaf(w2, w1, acc);
      }
    }
    out[idx] = acc;
  }
}

// fp32 [o][i][u][v] -> fp32 [u][v][i][o]
__global__ void k_pack_f32(const float *w, float *out, int c_out, int c_in, int k) {
  int total = c_out * c_in * k * k;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    int o = idx % c_out, i = (idx / c_out) % c_in, t = idx / (c_out * c_in);
    out[idx] = w[((size_t)o * c_in + i) * k * k + t];
  }
}

// depthwise fp32 [c][1][k][k] -> fp32 [k][k][c]
__global__ void k_pack_dw(const float *w, float *out, int c, int k) {
  int total = c * k * k;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    int ch = idx % c, t = idx / c;
    out[idx] = w[(size_t)ch * k * k + t];
  }
}

// fp32 [o][i][u][v] -> bf16 chunk planes [group][entry][n_pad][8] in the K order of KOrder
__global__ void k_pack_bf16(const float *w, __nv_bfloat16 *out, int c_out, KOrder ko) {
  const int total = ko.ng * ko.e_pad * ko.n_pad * 8;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    int c8 = idx % 8, o, plane;
    dc_packed_unchunk(ko, idx / 8, &plane, &o);
    int grp = plane / ko.e_pad, e = plane - grp * ko.e_pad;
    int pc, ccg, r, s;
    float v = 0.f;
    if (dc_korder_decode(ko, e, &pc, &ccg, &r, &s)) {
      if (ko.fold) {                       // row = (tap column, output channel)
        s = o / ko.co8;
        o -= s * ko.co8;
        if (s >= ko.k) o = c_out;          // padding rows
      } else if (ko.pair == 2) {           // row = (pixel of the pair, output channel); ccg = chunk of the pair row, s = shift
        const int elem = ccg * 8 + c8, ipx = elem / ko.c_in;
        const int px = o / ko.co8;
        o -= px * ko.co8;
        s = 2 * s + ipx - px;
        ccg = 0;
        c8 = elem - ipx * ko.c_in;         // channel (grp is 0 and cg irrelevant once ccg = 0)
        if (px >= 2 || s < 0 || s >= ko.k) o = c_out;
      } else if (ko.pair == 3) {           // stride 2: row = output channel; tap column = 2 * shift + pixel - (pad & 1)
        const int elem = ccg * 8 + c8, ipx = elem / ko.c_in;
        s = 2 * s + ipx - (ko.pad & 1);
        ccg = 0;
        c8 = elem - ipx * ko.c_in;
        if (s < 0 || s >= ko.k) o = c_out;
      }
      int c = (grp * ko.cg + ccg) * 8 + c8;
      if (o < c_out && c < ko.c_in) v = w[(((size_t)o * ko.c_in + c) * ko.k + r) * ko.k + s];
    }
    out[idx] = __float2bfloat16_rn(v);
  }
}

// Element (o, i, tap t) of the finished run as a dense kernel: a diagonal result is lifted, a
// pending identity is added.
__device__ __forceinline__ float merged_at(const Piece &p, int o, int i, int t) {
  const int kk = p.k * p.k, ctr = ((p.k - 1) / 2) * (p.k + 1);
  float w;
  if (p.diag) w = (o == i) ? p.w[(size_t)o * kk + t] : 0.f;
  else w = p.w[((size_t)o * p.c_in + i) * kk + t];
  if (p.ident && o == i && t == ctr) w += 1.f;
  return w;
}

// The bf16 packed copy with one thread per 16-byte chunk (8 input channels of one operand row),
// for large kernels (a thread walks eight elements, so small ones are faster element by element): the
// entry and row are decoded once per chunk, the eight weights are fetched by eight independent
// loads (an element that is padding reads element 0 and is then zeroed, so that no load sits behind
// a branch) and the chunk is written by one store.
__device__ __forceinline__ void deliver_packed_bf16_chunks(const Piece &acc, __nv_bfloat16 *out, const KOrder &ko,
                                                           int start, int stride) {
  const int c_out = acc.c_out, kk = acc.k * acc.k, ctr = ((acc.k - 1) / 2) * (acc.k + 1);
  const int total8 = ko.ng * ko.e_pad * ko.n_pad;
  for (int idx8 = start; idx8 < total8; idx8 += stride) {
    int plane, o_row;
    dc_packed_unchunk(ko, idx8, &plane, &o_row);
    const int grp = plane / ko.e_pad, e = plane - grp * ko.e_pad;
    int pc, ccg0, r, s0;
    bool live = dc_korder_decode(ko, e, &pc, &ccg0, &r, &s0);
    int o = o_row, px = 0;
    if (live) {
      if (ko.fold) {
        s0 = o / ko.co8;
        o -= s0 * ko.co8;
        if (s0 >= ko.k) live = false;
      } else if (ko.pair == 2) {
        px = o / ko.co8;
        o -= px * ko.co8;
        if (px >= 2) live = false;
      }
    }
    live = live && o < c_out;
    int ch[8], tap[8];
    bool ok[8];
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {
      int sx = s0, c;
      if (ko.pair >= 2) {
        const int elem = ccg0 * 8 + c8, ipx = elem / ko.c_in;
        sx = 2 * s0 + ipx - (ko.pair == 2 ? px : (ko.pad & 1));
        c = grp * ko.cg * 8 + elem - ipx * ko.c_in;
      } else {
        c = (grp * ko.cg + ccg0) * 8 + c8;
      }
      ok[c8] = live && sx >= 0 && sx < ko.k && c >= 0 && c < ko.c_in;
      ch[c8] = c;
      tap[c8] = r * ko.k + sx;
    }
    float w[8];
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {
      size_t off = 0;
      if (ok[c8]) off = acc.diag ? (size_t)o * kk + tap[c8] : ((size_t)o * acc.c_in + ch[c8]) * kk + tap[c8];
      w[c8] = acc.w[off];
    }
    __align__(16) __nv_bfloat16 v8[8];
#pragma unroll
    for (int c8 = 0; c8 < 8; ++c8) {
      float v = w[c8];
      if (acc.diag && o != ch[c8]) v = 0.f;
      if (acc.ident && o == ch[c8] && tap[c8] == ctr) v += 1.f;
      v8[c8] = __float2bfloat16_rn(ok[c8] ? v : 0.f);
    }
    *reinterpret_cast<uint4 *>(out + (size_t)idx8 * 8) = *reinterpret_cast<const uint4 *>(v8);
  }
}

// Last launch of a merge: writes the dense fp32 kernel (blocks [0, nb_w)), the bias (block nb_w)
// and, when asked for, the packed copy for the forward kernels (blocks after that; mode 1: fp32
// [u][v][i][o], mode 2: bf16 chunk planes in the K order of KOrder), all straight from the
// accumulated piece.
__global__ void k_deliver(Piece acc, float *w_merged, float *b_merged, void *packed, int mode, KOrder ko,
                          int nb_w, int nb_p, int chunked) {
  const int c_out = acc.c_out, c_in = acc.c_in, kk = acc.k * acc.k;
  int blk = (int)blockIdx.x;
  if (blk < nb_w) {
    const int total = c_out * c_in * kk;
    for (int idx = blk * blockDim.x + threadIdx.x; idx < total; idx += nb_w * blockDim.x) {
      const int t = idx % kk, i = (idx / kk) % c_in, o = idx / (kk * c_in);
      w_merged[idx] = merged_at(acc, o, i, t);
    }
    return;
  }
  blk -= nb_w;
  if (blk == 0) {
    for (int o = threadIdx.x; o < c_out; o += blockDim.x) b_merged[o] = acc.b[o];
    return;
  }
  blk -= 1;
  if (mode == 1) {
    float *out = reinterpret_cast<float *>(packed);
    const int total = c_out * c_in * kk;
    for (int idx = blk * blockDim.x + threadIdx.x; idx < total; idx += nb_p * blockDim.x) {
      const int o = idx % c_out, i = (idx / c_out) % c_in, t = idx / (c_out * c_in);
      out[idx] = merged_at(acc, o, i, t);
    }
  } else if (mode == 2 && chunked) {
    deliver_packed_bf16_chunks(acc, reinterpret_cast<__nv_bfloat16 *>(packed), ko, blk * blockDim.x + threadIdx.x,
                               nb_p * blockDim.x);
  } else if (mode == 2) {
    __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(packed);
    const int total = ko.ng * ko.e_pad * ko.n_pad * 8;
    for (int idx = blk * blockDim.x + threadIdx.x; idx < total; idx += nb_p * blockDim.x) {
      int c8 = idx % 8, o, plane;
      dc_packed_unchunk(ko, idx / 8, &plane, &o);
      int grp = plane / ko.e_pad, e = plane - grp * ko.e_pad;
      int pc, ccg, r, sx;
      float v = 0.f;
      if (dc_korder_decode(ko, e, &pc, &ccg, &r, &sx)) {
        if (ko.fold) {
          sx = o / ko.co8;
          o -= sx * ko.co8;
          if (sx >= ko.k) o = c_out;
        } else if (ko.pair == 2) {
          const int elem = ccg * 8 + c8, ipx = elem / ko.c_in;
          const int px = o / ko.co8;
          o -= px * ko.co8;
          sx = 2 * sx + ipx - px;
          ccg = 0;
          c8 = elem - ipx * ko.c_in;
          if (px >= 2 || sx < 0 || sx >= ko.k) o = c_out;
        } else if (ko.pair == 3) {
          const int elem = ccg * 8 + c8, ipx = elem / ko.c_in;
          sx = 2 * sx + ipx - (ko.pad & 1);
          ccg = 0;
          c8 = elem - ipx * ko.c_in;
          if (sx < 0 || sx >= ko.k) o = c_out;
        }
        const int c = (grp * ko.cg + ccg) * 8 + c8;
        if (o < c_out && c < ko.c_in) v = merged_at(acc, o, c, r * ko.k + sx);
      }
      out[idx] = __float2bfloat16_rn(v);
    }
  }
}

// ----------------------------------------------------------------------------------------------
// An inverted-residual block in one step: dense 1x1 (stride 1) -> depthwise k x k -> dense 1x1.
//
//   W'[o][i][t] = sum_c W3~[o][c] * D~[c][t] * W1~[c][i],   ~ = BN folded (scale g = gamma / sqrt(var + eps))
//   b'[o]       = b3~[o] + sum_c W3~[o][c] * (b2~[c] + (sum_t D~[c][t]) * b1~[c])
//
// which is what folding the three layers and composing them pairwise gives (Eq. 1 applied twice),
// without the folded copies and the 6x wider intermediate kernel ever going through global memory:
// each step of the pairwise walk waits for the one before, and for kernels of a few thousand
// elements those waits are the whole cost.  One CTA per output channel o; the raw layer weights are
// read once per CTA (they sit in L2), `chunk` hidden channels at a time.
// ----------------------------------------------------------------------------------------------
struct RawLayer {
  const float *w, *b, *gamma, *beta, *mean, *var;
  float eps;
};
struct BlockArgs {
  RawLayer l1, l2, l3;
  int c0, c1, c2, k;      // input, hidden, output channels; depthwise kernel size
  int chunk;              // hidden channels staged per pass
  float *w_out, *b_out;   // [c2][c0][k][k], [c2]
};
constexpr int kBlockThreads = 256;
constexpr int kBlockMaxPerThread = 8;       // outputs per thread: c0 * k * k <= 2048

__device__ __forceinline__ float raw_scale(const RawLayer &L, int o) {
  return L.gamma ? L.gamma[o] / sqrtf(L.var[o] + L.eps) : 1.f;
}
__device__ __forceinline__ float raw_bias(const RawLayer &L, int o, float g) {
  const float b = L.b ? L.b[o] : 0.f;
  return L.gamma ? fmaf(b - L.mean[o], g, L.beta[o]) : b;
}

// Up to kBlockBatch blocks of one run go out in one launch (blockIdx.y picks the block): they depend
// on the raw layers only, not on one another.
constexpr int kBlockBatch = 4;
struct BlockBatch {
  BlockArgs blk[kBlockBatch];
};

__global__ void __launch_bounds__(kBlockThreads) k_merge_block(const __grid_constant__ BlockBatch batch) {
  extern __shared__ __align__(16) float blk_smem[];
  const BlockArgs &a = batch.blk[blockIdx.y];
  if ((int)blockIdx.x >= a.c2) return;
  const int c0 = a.c0, c1 = a.c1, kk = a.k * a.k, J = c0 * kk, CH = a.chunk;
  float *Ms = blk_smem;                 // [CH][c0]  raw W1 rows
  float *Ds = Ms + CH * c0;             // [CH][kk]  raw D rows, then W3~[o][c] * D~[c][t] * g1[c]
  float *sc = Ds + CH * kk;             // [CH]      W3~[o][c] * g2[c] * g1[c]
  __shared__ float bias_part[kBlockThreads / 32];
  const int o = blockIdx.x, tid = threadIdx.x;
  const float g3 = raw_scale(a.l3, o);
  float acc[kBlockMaxPerThread];
  int oi[kBlockMaxPerThread], ot[kBlockMaxPerThread];
#pragma unroll
  for (int q = 0; q < kBlockMaxPerThread; ++q) {
    const int j = tid + q * kBlockThreads;
    acc[q] = 0.f;
    oi[q] = j / kk;
    ot[q] = j - oi[q] * kk;
  }
  float bsum = 0.f;
  for (int cb = 0; cb < c1; cb += CH) {
    const int rows = c1 - cb < CH ? c1 - cb : CH;
    // all loads of the pass go out together: W1 rows, D rows, and the per-channel scalars
    for (int e = tid; e < rows * c0; e += kBlockThreads) Ms[e] = a.l1.w[(size_t)cb * c0 + e];
    for (int e = tid; e < rows * kk; e += kBlockThreads) Ds[e] = a.l2.w[(size_t)cb * kk + e];
    for (int cl = tid; cl < rows; cl += kBlockThreads) {
      const int c = cb + cl;
      const float g1 = raw_scale(a.l1, c), g2 = raw_scale(a.l2, c);
      const float w3 = g3 * a.l3.w[(size_t)o * c1 + c];
      float dsum = 0.f;
      for (int t = 0; t < kk; ++t) dsum += g2 * a.l2.w[(size_t)c * kk + t];
      bsum = fmaf(w3, fmaf(dsum, raw_bias(a.l1, c, g1), raw_bias(a.l2, c, g2)), bsum);
      sc[cl] = (w3 * g2) * g1;
    }
    __syncthreads();
    for (int e = tid; e < rows * kk; e += kBlockThreads) Ds[e] *= sc[e / kk];
    __syncthreads();
#pragma unroll
    for (int q = 0; q < kBlockMaxPerThread; ++q) {
      if (tid + q * kBlockThreads < J) {
        const float *m = Ms + oi[q], *d = Ds + ot[q];
        float s = acc[q];
#pragma unroll 4
        for (int cl = 0; cl < rows; ++cl) s = fmaf(d[cl * kk], m[cl * c0], s);
        acc[q] = s;
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int q = 0; q < kBlockMaxPerThread; ++q) {
    const int j = tid + q * kBlockThreads;
    if (j < J) a.w_out[(size_t)o * J + j] = acc[q];
  }
  // bias: the per-thread terms meet through warp shuffles and one shared-memory hop
  for (int d = 16; d > 0; d >>= 1) bsum += __shfl_xor_sync(0xffffffffu, bsum, d);
  if ((tid & 31) == 0) bias_part[tid >> 5] = bsum;
  __syncthreads();
  if (tid == 0) {
    float b = 0.f;
    for (int w = 0; w < kBlockThreads / 32; ++w) b += bias_part[w];
    a.b_out[o] = raw_bias(a.l3, o, g3) + b;
  }
}

// ----------------------------------------------------------------------------------------------
// host: validation and geometry
// ----------------------------------------------------------------------------------------------

dc_status dc_validate_geom(const dc_geom *g) {
  if (!g) return DC_ERR_INVALID_ARG;
  if (g->c_in <= 0 || g->c_out <= 0 || g->k <= 0 || g->stride <= 0 || g->pad < 0 || g->groups <= 0)
    return DC_ERR_INVALID_ARG;
  if (g->k % 2 == 0) return DC_ERR_UNSUPPORTED;
  if (!(g->groups == 1 || (g->groups == g->c_in && g->c_in == g->c_out))) return DC_ERR_UNSUPPORTED;
  return DC_OK;
}

static dc_status validate_layer(const dc_layer *L) {
  dc_geom g = {L->c_in, L->c_out, L->groups, L->k, L->stride, L->pad};
  dc_status st = dc_validate_geom(&g);
  if (st != DC_OK) return st;
  if (!L->weight) return DC_ERR_INVALID_ARG;
  int nbn = (L->bn_gamma != nullptr) + (L->bn_beta != nullptr) + (L->bn_mean != nullptr) + (L->bn_var != nullptr);
  if (nbn != 0 && nbn != 4) return DC_ERR_INVALID_ARG;
  return DC_OK;
}

static size_t piece_elems(int c_in, int c_out, int k, int diag) {
  return diag ? (size_t)c_out * k * k : (size_t)c_out * c_in * k * k;
}

static int find_group(const dc_residual *res, int n_res, int first) {
  for (int i = 0; i < n_res; ++i)
    if (res[i].first == first) return i;
  return -1;
}

static dc_status check_chain(const dc_layer *layers, int n, const dc_residual *res, int n_res,
                             dc_geom *merged) {
  if (!layers || n <= 0 || n_res < 0 || (n_res > 0 && !res)) return DC_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    dc_status st = validate_layer(&layers[i]);
    if (st != DC_OK) return st;
    if (i > 0 && layers[i].c_in != layers[i - 1].c_out) return DC_ERR_SHAPE;
  }
  int prev_last = -1;
  for (int gi = 0; gi < n_res; ++gi) {
    if (res[gi].first < 0 || res[gi].last >= n || res[gi].first > res[gi].last) return DC_ERR_INVALID_ARG;
    if (res[gi].first <= prev_last) return DC_ERR_INVALID_ARG;
    prev_last = res[gi].last;
    int k = 1, s = 1, p = 0;
    for (int i = res[gi].first; i <= res[gi].last; ++i) {
      k += (layers[i].k - 1) * s;
      p += layers[i].pad * s;
      s *= layers[i].stride;
    }
    if (s != 1 || layers[res[gi].first].c_in != layers[res[gi].last].c_out || 2 * p != k - 1)
      return DC_ERR_NOT_MERGEABLE;
  }
  int k = 1, s = 1, p = 0;
  for (int i = 0; i < n; ++i) {
    k += (layers[i].k - 1) * s;
    p += layers[i].pad * s;
    s *= layers[i].stride;
  }
  if (merged) {
    merged->c_in = layers[0].c_in;
    merged->c_out = layers[n - 1].c_out;
    merged->groups = 1;
    merged->k = k; merged->stride = s; merged->pad = p;
  }
  return DC_OK;
}

// Bump allocator over the caller's workspace (256-byte granules); with base == nullptr it only counts.
struct Bump {
  char *base; size_t off;
  float *take(size_t elems) {
    size_t bytes = dc_round_up(elems * sizeof(float), 256);
    float *p = base ? reinterpret_cast<float *>(base + off) : nullptr;
    off += bytes;
    return p;
  }
};

static inline int blocks_for(size_t total, int threads) {
  size_t b = (total + threads - 1) / threads;
  return (int)(b > 65535 ? 65535 : (b == 0 ? 1 : b));
}

// Composes second o first into a new piece; launches when `go`.
static Piece compose(const Piece &first, const Piece &second, Bump &bump, bool go, cudaStream_t st) {
  Piece out;
  out.c_in = first.c_in; out.c_out = second.c_out;
  out.k = first.k + (second.k - 1) * first.stride;
  out.stride = first.stride * second.stride;
  out.diag = first.diag && second.diag;
  out.ident = 0;
  size_t elems = piece_elems(out.c_in, out.c_out, out.k, out.diag);
  float *w = bump.take(elems);
  float *b = bump.take(out.c_out);
  out.w = w; out.b = b;
  if (go) {
    const int nbias = bias_blocks(out.c_out, 256);
    if (!first.diag && !second.diag && first.k == 1 && first.stride == 1 && second.k > 1 &&
        first.c_out * second.k * second.k <= kAfter1x1MaxFloats) {
      dim3 grid(dc_div_up(out.c_in * out.k * out.k, 256), out.c_out + 1);
      if ((int)grid.x < nbias) grid.x = nbias;
      k_compose_after_1x1<<<grid, 256, 0, st>>>(first, second, w, b);
    } else if (!first.diag && !second.diag && elems <= (size_t)200000 && second.k <= 7) {
      const int gx = dc_div_up(out.c_in * out.k * out.k, 32), gy = dc_div_up(out.c_out, 8);
      k_compose_dd_small<<<gx * gy + nbias, 256, 0, st>>>(first, second, w, b, out.k, gx, gy);
    } else if (!first.diag && !second.diag && first.k == 3 && second.k == 3 && first.stride == 1) {
      const int gx = dc_div_up(out.c_in, 32), gy = dc_div_up(out.c_out, 16);
      k_compose_poly33<<<gx * gy + nbias, 256, 0, st>>>(first, second, w, b, gx, gy);
    } else if (!first.diag && !second.diag) {
      // 128 x 64 tiles when they still give every SM two tiles, 64 x 64 otherwise
      const int gx = dc_div_up(out.c_in * out.k * out.k, 64);
      const int gy8 = dc_div_up(out.c_out, 128), gy4 = dc_div_up(out.c_out, 64);
      if (gx * gy8 >= 2 * dc_sm_count())
        k_compose_dd_tiled<8><<<gx * gy8 + nbias, 256, 0, st>>>(first, second, w, b, out.k, gx, gy8);
      else
        k_compose_dd_tiled<4><<<gx * gy4 + nbias, 256, 0, st>>>(first, second, w, b, out.k, gx, gy4);
    } else {
      const int nb = blocks_for(elems, 256);
      k_compose_diag<<<nb + nbias, 256, 0, st>>>(first, second, w, b, out.k, (int)elems, nb);
    }
  }
  return out;
}

// Index of the skip group that contains layer idx, or -1.
static int group_of(const dc_residual *res, int n_res, int idx) {
  for (int i = 0; i < n_res; ++i)
    if (res[i].first <= idx && idx <= res[i].last) return i;
  return -1;
}

// Hidden channels k_merge_block stages per pass for this block (0: the block does not qualify).
static int block_chunk(const dc_layer *L, int n, const dc_residual *res, int n_res, int i) {
  if (i + 2 >= n) return 0;
  const dc_layer &e = L[i], &d = L[i + 1], &p = L[i + 2];
  if (e.groups != 1 || e.k != 1 || e.stride != 1 || e.pad != 0) return 0;
  if (d.groups == 1 || d.groups != d.c_in) return 0;
  if (p.groups != 1 || p.k != 1 || p.stride != 1 || p.pad != 0) return 0;
  if (e.c_in * d.k * d.k > kBlockThreads * kBlockMaxPerThread) return 0;
  // wide blocks are faster step by step: their compositions fill the GPU, one CTA per output channel does not
  if ((long)e.c_out * e.c_in * d.k * d.k > 150000) return 0;
  const int g0 = group_of(res, n_res, i), g1 = group_of(res, n_res, i + 1), g2 = group_of(res, n_res, i + 2);
  const bool whole = g0 >= 0 && g0 == g1 && g1 == g2 && res[g0].first == i && res[g0].last == i + 2;
  if (!whole && (g0 >= 0 || g1 >= 0 || g2 >= 0)) return 0;
  const int per = e.c_in + d.k * d.k + 1;
  int ch = (200 * 1024 / 4) / per;
  if (ch > e.c_out) ch = e.c_out;
  return ch >= 32 || ch == e.c_out ? ch : 0;
}

static RawLayer raw_of(const dc_layer &L) {
  return RawLayer{L.weight, L.bias, L.bn_gamma, L.bn_beta, L.bn_mean, L.bn_var, L.bn_eps};
}

// One walk drives both the size query (go == false: nothing is dereferenced or launched) and the
// launches (go == true: the caller has already checked workspace_bytes against the query).
static dc_status merge_walk(const dc_layer *layers, int n, const dc_residual *res, int n_res,
                            float *w_merged, float *b_merged, void *w_packed, dc_dtype packed_dtype,
                            void *workspace, cudaStream_t st, bool go, dc_geom *merged, size_t *need,
                            dc_merge_algo algo = DC_MERGE_AUTO) {
  dc_geom mg;
  dc_status s = check_chain(layers, n, res, n_res, &mg);
  if (s != DC_OK) return s;
  if (merged) *merged = mg;
  Bump bump{go ? (char *)workspace : nullptr, 0};

  // 0. inverted-residual blocks (1x1, depthwise, 1x1) are merged in one step from the raw layers
  std::vector<int> chunk_at(n, 0), covered(n, 0);
  if (algo != DC_MERGE_STEPS)
    for (int i = 0; i + 2 < n;) {
      const int ch = block_chunk(layers, n, res, n_res, i);
      if (ch > 0) { chunk_at[i] = ch; covered[i] = covered[i + 1] = covered[i + 2] = 1; i += 3; }
      else ++i;
    }

  // 1. fold every other layer
  std::vector<Piece> folded(n);
  {
    FoldTable t;
    int cnt = 0;
    size_t max_total = 1;
    auto flush = [&]() {
      if (cnt == 0) return;
      t.n = cnt;
      if (go) {
        int bx = blocks_for(max_total, 256);
        dim3 grid(bx > 1024 ? 1024 : bx, cnt);       // a few elements per thread: the launch is short beside its chain
        k_fold_bn<<<grid, 256, 0, st>>>(t);
      }
      cnt = 0;
      max_total = 1;
    };
    for (int l = 0; l < n; ++l) {
      if (covered[l]) continue;
      const dc_layer &L = layers[l];
      int diag = L.groups != 1;
      size_t elems = piece_elems(L.c_in, L.c_out, L.k, diag);
      float *w = bump.take(elems), *b = bump.take(L.c_out);
      t.w[cnt] = L.weight; t.b[cnt] = L.bias; t.gamma[cnt] = L.bn_gamma; t.beta[cnt] = L.bn_beta;
      t.mean[cnt] = L.bn_mean; t.var[cnt] = L.bn_var; t.eps[cnt] = L.bn_eps;
      t.w_out[cnt] = w; t.b_out[cnt] = b;
      t.c_out[cnt] = L.c_out; t.per_out[cnt] = (int)(elems / L.c_out);
      if (elems > max_total) max_total = elems;
      folded[l] = Piece{w, b, L.c_in, L.c_out, L.k, L.stride, diag, 0};
      if (++cnt == DC_FOLD_MAX) flush();
    }
    flush();
  }

  // 2. compose: blocks and skip groups first (with their identity tap), then left to right
  BlockBatch batch;
  int n_batch = 0, batch_grid = 0;
  size_t batch_smem = 0;
  auto flush_blocks = [&]() {
    if (n_batch == 0) return;
    static unsigned char attr_done[kDcMaxDevices];
    dc_set_max_smem_once(k_merge_block, 200 * 1024, attr_done);
    k_merge_block<<<dim3(batch_grid, n_batch), kBlockThreads, batch_smem, st>>>(batch);
    n_batch = 0; batch_grid = 0; batch_smem = 0;
  };
  Piece acc{};
  bool have = false;
  int i = 0;
  while (i < n) {
    Piece piece;
    int gi = find_group(res, n_res, i);
    if (chunk_at[i] > 0) {
      const dc_layer &e = layers[i], &d = layers[i + 1], &p = layers[i + 2];
      piece = Piece{nullptr, nullptr, e.c_in, p.c_out, d.k, d.stride, 0, gi >= 0 ? 1 : 0};
      float *w = bump.take(piece_elems(piece.c_in, piece.c_out, piece.k, 0));
      float *b = bump.take(piece.c_out);
      piece.w = w; piece.b = b;
      if (go) {
        batch.blk[n_batch] = BlockArgs{raw_of(e), raw_of(d), raw_of(p), e.c_in, e.c_out, p.c_out, d.k, chunk_at[i], w, b};
        const size_t smem = (size_t)chunk_at[i] * (e.c_in + d.k * d.k + 1) * sizeof(float);
        if (smem > batch_smem) batch_smem = smem;
        if (p.c_out > batch_grid) batch_grid = p.c_out;
        // the blocks read raw layers only: hold the launch until the batch is full or a composition
        // needs one of its pieces
        if (++n_batch == kBlockBatch) flush_blocks();
      }
      i += 3;
    } else if (gi < 0) {
      piece = folded[i];
      ++i;
    } else {
      piece = folded[res[gi].first];
      if (go) flush_blocks();
      for (int j = res[gi].first + 1; j <= res[gi].last; ++j) piece = compose(piece, folded[j], bump, go, st);
      piece.ident = 1;          // f(x) + x: the identity kernel rides along as a flag
      i = res[gi].last + 1;
    }
    if (!have) { acc = piece; have = true; }
    else {
      if (go) flush_blocks();
      acc = compose(acc, piece, bump, go, st);
    }
  }
  if (need) *need = bump.off + 256;
  if (!go) return DC_OK;
  flush_blocks();

  // 3. deliver: dense fp32 result, bias, optional packed copy, in one launch
  size_t elems = (size_t)mg.c_out * mg.c_in * mg.k * mg.k;
  KOrder ko;
  dc_korder_init(&ko, &mg);
  int mode = 0;
  size_t p_elems = 0;
  if (w_packed) {
    mode = packed_dtype == DC_F32 ? 1 : 2;
    p_elems = mode == 1 ? elems : (size_t)ko.ng * ko.e_pad * ko.n_pad * 8;
    if (!dc_aligned16(w_packed)) return DC_ERR_ALIGNMENT;
  }
  const int chunked = mode == 2 && p_elems >= (size_t)262144;
  const int nb_w = blocks_for(elems, 256), nb_p = mode ? blocks_for(chunked ? p_elems / 8 : p_elems, 256) : 0;
  k_deliver<<<nb_w + 1 + nb_p, 256, 0, st>>>(acc, w_merged, b_merged, w_packed, mode, ko, nb_w, nb_p, chunked);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

// Workspace bytes that cover either launch form.
static dc_status merge_need(const dc_layer *layers, int n, const dc_residual *res, int n_res, dc_geom *merged,
                            size_t *need) {
  size_t a = 0, b = 0;
  dc_status s = merge_walk(layers, n, res, n_res, nullptr, nullptr, nullptr, DC_F32, nullptr, nullptr, false, merged,
                           &a, DC_MERGE_AUTO);
  if (s != DC_OK) return s;
  s = merge_walk(layers, n, res, n_res, nullptr, nullptr, nullptr, DC_F32, nullptr, nullptr, false, nullptr, &b,
                 DC_MERGE_STEPS);
  if (s != DC_OK) return s;
  if (need) *need = a > b ? a : b;
  return DC_OK;
}

// ----------------------------------------------------------------------------------------------
// exported
// ----------------------------------------------------------------------------------------------

extern "C" dc_status dc_fold_bn(const dc_layer *layer, float *w_out, float *b_out, dc_stream stream) {
  if (!layer || !w_out || !b_out) return DC_ERR_INVALID_ARG;
  dc_status s = validate_layer(layer);
  if (s != DC_OK) return s;
  if (!dc_aligned16(layer->weight) || !dc_aligned16(w_out) || !dc_aligned16(b_out)) return DC_ERR_ALIGNMENT;
  FoldTable t;
  t.n = 1;
  size_t elems = piece_elems(layer->c_in, layer->c_out, layer->k, layer->groups != 1);
  t.w[0] = layer->weight; t.b[0] = layer->bias; t.gamma[0] = layer->bn_gamma; t.beta[0] = layer->bn_beta;
  t.mean[0] = layer->bn_mean; t.var[0] = layer->bn_var; t.eps[0] = layer->bn_eps;
  t.w_out[0] = w_out; t.b_out[0] = b_out; t.c_out[0] = layer->c_out; t.per_out[0] = (int)(elems / layer->c_out);
  int bx = blocks_for(elems, 256);
  dim3 grid(bx > 256 ? 256 : bx, 1);
  k_fold_bn<<<grid, 256, 0, (cudaStream_t)stream>>>(t);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

extern "C" dc_status dc_merge_query(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                                    dc_geom *merged, size_t *workspace_bytes) {
  return merge_need(layers, n_layers, res, n_res, merged, workspace_bytes);
}

extern "C" dc_status dc_merge_chain_algo(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                                         float *w_merged, float *b_merged, void *w_packed, dc_dtype packed_dtype,
                                         void *workspace, size_t workspace_bytes, dc_stream stream,
                                         dc_merge_algo algo) {
  if (!w_merged || !b_merged) return DC_ERR_INVALID_ARG;
  if (packed_dtype != DC_F32 && packed_dtype != DC_BF16) return DC_ERR_INVALID_ARG;
  if (algo != DC_MERGE_AUTO && algo != DC_MERGE_STEPS) return DC_ERR_INVALID_ARG;
  size_t need = 0;
  dc_status s = merge_need(layers, n_layers, res, n_res, nullptr, &need);
  if (s != DC_OK) return s;
  if (!workspace || workspace_bytes < need) return DC_ERR_WORKSPACE;
  if (!dc_aligned16(w_merged) || !dc_aligned16(b_merged) || !dc_aligned16(workspace) ||
      (w_packed && !dc_aligned16(w_packed)))
    return DC_ERR_ALIGNMENT;
  for (int i = 0; i < n_layers; ++i)
    if (!dc_aligned16(layers[i].weight)) return DC_ERR_ALIGNMENT;
  return merge_walk(layers, n_layers, res, n_res, w_merged, b_merged, w_packed, packed_dtype, workspace,
                    (cudaStream_t)stream, true, nullptr, nullptr, algo);
}

extern "C" dc_status dc_merge_chain(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                                    float *w_merged, float *b_merged, void *w_packed, dc_dtype packed_dtype,
                                    void *workspace, size_t workspace_bytes, dc_stream stream) {
  return dc_merge_chain_algo(layers, n_layers, res, n_res, w_merged, b_merged, w_packed, packed_dtype, workspace,
                             workspace_bytes, stream, DC_MERGE_AUTO);
}

extern "C" dc_status dc_packed_bytes(const dc_geom *g, dc_dtype dtype, size_t *bytes) {
  dc_status s = dc_validate_geom(g);
  if (s != DC_OK) return s;
  if (!bytes || (dtype != DC_F32 && dtype != DC_BF16)) return DC_ERR_INVALID_ARG;
  if (g->groups != 1) { *bytes = (size_t)g->c_out * g->k * g->k * sizeof(float); return DC_OK; }
  if (dtype == DC_F32) { *bytes = (size_t)g->c_out * g->c_in * g->k * g->k * sizeof(float); return DC_OK; }
  KOrder ko;
  dc_korder_init(&ko, g);
  *bytes = (size_t)ko.ng * ko.e_pad * ko.n_pad * 8 * sizeof(__nv_bfloat16);
  return DC_OK;
}

extern "C" dc_status dc_pack_weights(const float *w, const dc_geom *g, dc_dtype dtype, void *w_packed,
                                     dc_stream stream) {
  dc_status s = dc_validate_geom(g);
  if (s != DC_OK) return s;
  if (!w || !w_packed || (dtype != DC_F32 && dtype != DC_BF16)) return DC_ERR_INVALID_ARG;
  if (!dc_aligned16(w) || !dc_aligned16(w_packed)) return DC_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  if (g->groups != 1) {
    size_t total = (size_t)g->c_out * g->k * g->k;
    k_pack_dw<<<blocks_for(total, 256), 256, 0, st>>>(w, (float *)w_packed, g->c_out, g->k);
  } else if (dtype == DC_F32) {
    size_t total = (size_t)g->c_out * g->c_in * g->k * g->k;
    k_pack_f32<<<blocks_for(total, 256), 256, 0, st>>>(w, (float *)w_packed, g->c_out, g->c_in, g->k);
  } else {
    KOrder ko;
    dc_korder_init(&ko, g);
    size_t total = (size_t)ko.ng * ko.e_pad * ko.n_pad * 8;
    k_pack_bf16<<<blocks_for(total, 256), 256, 0, st>>>(w, (__nv_bfloat16 *)w_packed, g->c_out, ko);
  }
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}

// ----------------------------------------------------------------------------------------------
// Merge without any caller-provided or allocated scratch memory.
//
// Some callers cannot allocate device memory at the point where they merge: code running inside a
// memory-pool or allocator callback, a plug-in whose host forbids allocation calls after
// initialisation, or a process that has handed the whole GPU to another allocator.  For them the
// intermediate kernels of the merge live in a fixed array that is part of the library image: every
// GPU that loads the library holds these bytes until the process exits.
// ----------------------------------------------------------------------------------------------
#define DC_STATIC_SCRATCH_BYTES (4u << 20)
static __device__ __align__(256) unsigned char g_merge_scratch[DC_STATIC_SCRATCH_BYTES];

// In host code the symbol above is only a handle; the device address is looked up once per device.
#define DC_MAX_DEVICES 64
static void *g_merge_scratch_addr[DC_MAX_DEVICES];

extern "C" size_t dc_merge_chain_static_capacity(void) { return (size_t)DC_STATIC_SCRATCH_BYTES; }

extern "C" dc_status dc_merge_chain_static(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                                           float *w_merged, float *b_merged, void *w_packed,
                                           dc_dtype packed_dtype, dc_stream stream) {
  if (!w_merged || !b_merged) return DC_ERR_INVALID_ARG;
  if (packed_dtype != DC_F32 && packed_dtype != DC_BF16) return DC_ERR_INVALID_ARG;
  size_t need = 0;
  dc_status s = merge_need(layers, n_layers, res, n_res, nullptr, &need);
  if (s != DC_OK) return s;
  if (need > (size_t)DC_STATIC_SCRATCH_BYTES) return DC_ERR_WORKSPACE;   // run too large for the built-in scratch
  if (!dc_aligned16(w_merged) || !dc_aligned16(b_merged) || (w_packed && !dc_aligned16(w_packed)))
    return DC_ERR_ALIGNMENT;
  for (int i = 0; i < n_layers; ++i)
    if (!dc_aligned16(layers[i].weight)) return DC_ERR_ALIGNMENT;
  int dev = -1;
  DC_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= DC_MAX_DEVICES) return DC_ERR_UNSUPPORTED;
  if (!g_merge_scratch_addr[dev]) {
    // first call on this device (with that device current): resolve the array's device address
    void *ptr = nullptr;
    DC_CUDA_OK(cudaGetSymbolAddress(&ptr, g_merge_scratch));
    if (!ptr) return DC_ERR_CUDA;
    g_merge_scratch_addr[dev] = ptr;
  }
  // Nothing in the scratch has to start at zero: every intermediate is written in full before it
  // is read, so the contents a previous call left behind are simply overwritten.
  return merge_walk(layers, n_layers, res, n_res, w_merged, b_merged, w_packed, packed_dtype,
                    g_merge_scratch_addr[dev], (cudaStream_t)stream, true, nullptr, nullptr);
}
