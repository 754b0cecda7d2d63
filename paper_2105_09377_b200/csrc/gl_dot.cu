// gl_cartesian_dot: compute dotProd (cartProd (windows? a0) a1)   (Fig. 2a, 2b, Fig. 6)
//
// The pairing that cartProd describes (Section 4.2) is never stored: it is the
// pairing of an A tile with a B tile inside a GEMM  out[m,o] = sum_k A[m,k] B[o,k].
// Tensor-core path (sm_100a):
//   * operands are staged in shared memory by TMA.  For a convolution the rows
//     of A are windows of a channels-last activation tensor and the TMA unit
//     forms them itself (im2col tensor map: window origin, filter offset, zero
//     fill outside the image), so the im2col matrix of Section 5.3 never exists;
//   * tcgen05.mma (bf16 x bf16 -> fp32) issued by one thread accumulates into
//     TMEM; two accumulator buffers let the epilogue of one tile overlap the
//     main loop of the next;
//   * four epilogue warps read TMEM with tcgen05.ld, apply relu if asked and
//     store fp32 rows.
// A general SIMT kernel covers every other shape (odd K, arbitrary-rank windows).
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <mutex>
#include <string>
#include <unordered_map>

#include "gl_internal.h"
#include "gl_launch.cuh"

using namespace gl;

namespace {

__device__ unsigned int g_status = 0;   // sticky: set when a bounded wait gives up



// ------------------------------------------------------------------------
// General SIMT kernel
// ------------------------------------------------------------------------

struct GenA {            // how to fetch A[m,k]
  int mode;              // 0 plain [M,K]; 1 conv windows; 2 arbitrary windows
  int64_t M, K, O;
  // conv
  int channels_last;
  int64_t C, H, W, Kh, Kw, Sh, Sw, ph, pw, Ho, Wo;
  // arbitrary windows
  int n;
  int64_t in_size[GL_MAX_DIMS], in_stride[GL_MAX_DIMS], out_ext[GL_MAX_DIMS];
  int64_t w[GL_MAX_DIMS], s[GL_MAX_DIMS], pad_lo[GL_MAX_DIMS];
  int64_t item;
  // result layout: [M,O], or (image, O, H'W') when the squeeze + transpose of Fig. 2a is fused
  int out_nchw;
  int out_bf16;   // results rounded to bf16 (nearest even) and stored as 2-byte elements
  int64_t HoWo;
};

__device__ __forceinline__ float bf16_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }
// Two fp32 values (as bits) rounded to nearest-even bf16 and packed: `lo` at the lower address.
__device__ __forceinline__ uint32_t pack_bf16x2(uint32_t lo, uint32_t hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(__uint_as_float(hi)), "f"(__uint_as_float(lo)));
  return d;
}
__device__ __forceinline__ uint16_t f32_to_bf16(float v) { return static_cast<uint16_t>(pack_bf16x2(__float_as_uint(v), 0u) & 0xFFFFu); }

__device__ float fetch_a(const uint16_t* __restrict__ a, const GenA& g, int64_t m, int64_t k) {
  if (g.mode == 0) return bf16_to_f32(a[m * g.K + k]);
  if (g.mode == 1) {
    const int64_t wo = m % g.Wo, ho = (m / g.Wo) % g.Ho, n = m / (g.Wo * g.Ho);
    int64_t c, kh, kw;
    if (g.channels_last) { c = k % g.C; kw = (k / g.C) % g.Kw; kh = k / (g.C * g.Kw); }
    else { kw = k % g.Kw; kh = (k / g.Kw) % g.Kh; c = k / (g.Kw * g.Kh); }
    const int64_t h = ho * g.Sh + kh - g.ph, w = wo * g.Sw + kw - g.pw;
    if (h < 0 || h >= g.H || w < 0 || w >= g.W) return 0.f;
    const int64_t off = g.channels_last ? ((n * g.H + h) * g.W + w) * g.C + c : ((n * g.C + c) * g.H + h) * g.W + w;
    return bf16_to_f32(a[off]);
  }
  int64_t q[GL_MAX_DIMS], idx = k, off = 0;
  for (int d = g.n - 1; d >= 0; --d) { q[d] = idx % g.w[d]; idx /= g.w[d]; }
  idx = m;
  bool inside = true;
  for (int d = g.n - 1; d >= 0; --d) {
    const int64_t pos = (idx % g.out_ext[d]) * g.s[d] + q[d] - g.pad_lo[d];
    idx /= g.out_ext[d];
    inside = inside && pos >= 0 && pos < g.in_size[d];
    off += pos * g.in_stride[d];
  }
  return inside ? bf16_to_f32(a[idx * g.item + off]) : 0.f;
}

// 64x64 output tile per block, 4x4 per thread, K in steps of 16.
__global__ void __launch_bounds__(256) dot_general(const uint16_t* __restrict__ a, const uint16_t* __restrict__ b,
                                                   float* __restrict__ out, const GenA g, int relu) {
  __shared__ float sa[16][64 + 1], sb[16][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t m0 = (int64_t)blockIdx.x * 64, o0 = (int64_t)blockIdx.y * 64;
  float acc[4][4] = {};
  for (int64_t k0 = 0; k0 < g.K; k0 += 16) {
    for (int e = threadIdx.x; e < 16 * 64; e += 256) {
      const int kk = e & 15, r = e >> 4;
      const int64_t k = k0 + kk;
      sa[kk][r] = (m0 + r < g.M && k < g.K) ? fetch_a(a, g, m0 + r, k) : 0.f;
      sb[kk][r] = (o0 + r < g.O && k < g.K) ? bf16_to_f32(b[(o0 + r) * g.K + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = sa[kk][ty * 4 + i]; bv[i] = sb[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t m = m0 + ty * 4 + i, o = o0 + tx * 4 + j;
      if (m < g.M && o < g.O) {
        float v = acc[i][j];
        if (relu) v = v > 0.f ? v : 0.f;
        const int64_t at = g.out_nchw ? ((m / g.HoWo) * g.O + o) * g.HoWo + m % g.HoWo : m * g.O + o;
        if (g.out_bf16) reinterpret_cast<uint16_t*>(out)[at] = f32_to_bf16(v);
        else out[at] = v;
      }
    }
}

// ------------------------------------------------------------------------
// Layout pre-pass for the paper's (C,H,W) item layout: channels-last copies
// with the channel count padded to a multiple of 8 (16 bytes of bf16), which
// is what the TMA unit can address.
// ------------------------------------------------------------------------

// X (N,C,HW) -> (N,HW,Cp), zero for c >= C.
__global__ void __launch_bounds__(256) nchw_to_nhwc_pad(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                                        int64_t C, int64_t HW, int64_t Cp) {
  __shared__ uint16_t tile[32][34];
  const int64_t n = blockIdx.z, c0 = (int64_t)blockIdx.y * 32, p0 = (int64_t)blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t c = c0 + ty + 8 * i, p = p0 + tx;
    tile[ty + 8 * i][tx] = (c < C && p < HW) ? in[(n * C + c) * HW + p] : (uint16_t)0;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t p = p0 + ty + 8 * i, c = c0 + tx;
    if (p < HW && c < Cp) out[(n * HW + p) * Cp + c] = tile[tx][ty + 8 * i];
  }
}

// W (O,C,T) -> (O,T,Cp) with T = Kh*Kw, zero for c >= C.
__global__ void __launch_bounds__(256) weights_to_channels_last(const uint16_t* __restrict__ in,
                                                                uint16_t* __restrict__ out, int64_t O, int64_t C,
                                                                int64_t T, int64_t Cp) {
  const int64_t total = O * T * Cp;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t c = e % Cp, t = (e / Cp) % T, o = e / (Cp * T);
    out[e] = c < C ? in[(o * C + c) * T + t] : (uint16_t)0;
  }
}

// Both layout copies of a (C,H,W)-item convolution in ONE launch.
// Blocks [0, x_blocks): activations (N,C,H,W) -> (N,Hs,Ws,Cp), channels padded with zeros to Cp.  (Hs,Ws) is
// the whole image, or - for 1x1 windows without padding, which touch only every (Sh,Sw)-th pixel - just
// those pixels, so that the copy is the [N*H'*W', Cp] matrix itself.  A block moves 64 pixels (counted
// across images, so that small images leave no ragged tiles) x 64 channels: pixel-contiguous reads, 16-byte
// channel-contiguous writes.
// Blocks from x_blocks on: weights (O,C,T) -> (O,T,Cp), T = Kh*Kw; a WARP takes 64 channels x T taps of one
// filter: one contiguous run read with 16-byte loads, T runs of 64 channels written as 16-byte pieces.
struct PrepassParams {
  int C, H, W, Cp, Hs, Ws, Sh, Sw;
  int tiles_c, x_blocks;            // channel tiles; activation blocks = pixel tiles * tiles_c
  int64_t total_pix;                // N * Hs * Ws
  int O, T, wtiles_c, wwarps;       // weight units = O * wtiles_c, wwarps of them per block
  int fast;                         // total_pix + 64 < 2^31: pixel indices divide by multiply-high
  FastDiv by_tiles_c, by_npix, by_Ws;
};

__global__ void __launch_bounds__(256) nchw_prepass(const uint16_t* __restrict__ x, uint16_t* __restrict__ xs,
                                                    const uint16_t* __restrict__ w, uint16_t* __restrict__ ws,
                                                    const PrepassParams p) {
  extern __shared__ uint16_t pre_smem[];
  int b = blockIdx.x;
  // While the predecessor drains, an activation block requests the lines of its loads into L2 (a prefetch
  // consumes nothing; a line that is still being written is updated in L2, where all writes meet).
  if (b < p.x_blocks) {
    const int pt0 = static_cast<int>(fdiv(static_cast<uint32_t>(b), p.by_tiles_c));
    const int c00 = (b - pt0 * p.tiles_c) * 64;
    const int npix0 = p.Hs * p.Ws;
    const int64_t HW0 = static_cast<int64_t>(p.H) * p.W;
    // one line per (channel, 32-pixel stretch): thread t takes channel t / 4 and stretch t % 4 of the tile's 64
    // pixels (for strided windows the stretch covers Sw times as many input pixels: two lines)
    const int ch = threadIdx.x >> 2, part = threadIdx.x & 3;
    const int64_t gp = static_cast<int64_t>(pt0) * 64 + 16 * part;
    if (gp < p.total_pix && c00 + ch < p.C) {
      const int64_t n = p.fast ? static_cast<int64_t>(fdiv(static_cast<uint32_t>(gp), p.by_npix)) : gp / npix0;
      const int pix = static_cast<int>(gp - n * npix0);
      const int hs = static_cast<int>(fdiv(static_cast<uint32_t>(pix), p.by_Ws)), wsx = pix - hs * p.Ws;
      const uint16_t* at = x + (n * p.C + c00 + ch) * HW0 + static_cast<int64_t>(hs) * p.Sh * p.W + wsx * p.Sw;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(at) : "memory");
    }
  }
  pdl_wait();
  pdl_launch_dependents();
  if (b >= p.x_blocks) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (wid >= p.wwarps) return;
    const int unit = (b - p.x_blocks) * p.wwarps + wid;
    if (unit >= p.O * p.wtiles_c) return;
    const int o = unit / p.wtiles_c, c0 = (unit - o * p.wtiles_c) * 64;
    const int nc = max(0, min(64, p.C - c0));   // channels with data (none in a fully padded tail)
    const int run = nc * p.T;                    // contiguous elements of this filter and channel tile
    const uint16_t* src = w + (static_cast<int64_t>(o) * p.C + c0) * p.T;
    uint16_t* mine = pre_smem + wid * 64 * p.T;
    const bool vec_in = (reinterpret_cast<uintptr_t>(src) & 15u) == 0;
    const int nvec = vec_in ? run >> 3 : 0;
    for (int v = lane; v < nvec; v += 32) reinterpret_cast<uint4*>(mine)[v] = reinterpret_cast<const uint4*>(src)[v];
    for (int e = nvec * 8 + lane; e < run; e += 32) mine[e] = src[e];
    __syncwarp();
    // output pieces: tap t, channels c0 + 8 g .. + 7; channels past C are zeros
    const int groups = (min(64, p.Cp - c0) + 7) >> 3;
    for (int piece = lane; piece < p.T * 8; piece += 32) {
      const int t = piece >> 3, g = piece & 7;
      if (g < groups) {
        uint32_t wd[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int ca = g * 8 + 2 * i, cb = ca + 1;
          const uint32_t lo = ca < nc ? mine[ca * p.T + t] : 0u, hi = cb < nc ? mine[cb * p.T + t] : 0u;
          wd[i] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4*>(ws + (static_cast<int64_t>(o) * p.T + t) * p.Cp + c0 + g * 8) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
      }
    }
    return;
  }
  constexpr int kPitch = 66;                 // elements per staged channel row
  const int pt = static_cast<int>(fdiv(static_cast<uint32_t>(b), p.by_tiles_c));   // pixel tile
  const int tc = b - pt * p.tiles_c;
  const int64_t g0 = static_cast<int64_t>(pt) * 64;   // first pixel of the tile, counted over all images
  const int c0 = tc * 64;
  const int npix = p.Hs * p.Ws;
  const int64_t HW = static_cast<int64_t>(p.H) * p.W;
  // reads.  Whole images with a pixel count that is a multiple of 4: a thread loads 4 consecutive pixels
  // (8 bytes) of 4 channels.  Otherwise: a warp takes one channel, its lanes two stretches of 32 pixels.
  const bool wide = p.Sh == 1 && p.Sw == 1 && p.Hs == p.H && p.Ws == p.W && (npix & 3) == 0 &&
                    (reinterpret_cast<uintptr_t>(x) & 7u) == 0;
  if (wide) {
    const int pg = threadIdx.x & 15, cs = threadIdx.x >> 4;
    const int64_t gp = g0 + 4 * pg;
    const bool pok = gp < p.total_pix;
    const int64_t n = p.fast ? static_cast<int64_t>(fdiv(static_cast<uint32_t>(gp), p.by_npix)) : gp / npix;
    const uint16_t* src = x + (n * p.C + c0 + cs) * HW + (gp - n * npix);
    uint2 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[i] = make_uint2(0u, 0u);
      if (pok && c0 + cs + 16 * i < p.C) v[i] = *reinterpret_cast<const uint2*>(src + 16 * i * HW);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t* dst = reinterpret_cast<uint32_t*>(pre_smem + (cs + 16 * i) * kPitch + 4 * pg);
      dst[0] = v[i].x;
      dst[1] = v[i].y;
    }
  } else {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint16_t* src[2];
    bool pok[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int64_t gp = g0 + j * 32 + lane;
      pok[j] = gp < p.total_pix;
      const int64_t n = p.fast ? static_cast<int64_t>(fdiv(static_cast<uint32_t>(gp), p.by_npix)) : gp / npix;
      const int pix = static_cast<int>(gp - n * npix);
      const int hs = static_cast<int>(fdiv(static_cast<uint32_t>(pix), p.by_Ws)), wsx = pix - hs * p.Ws;
      src[j] = x + (n * p.C + c0 + wid) * HW + hs * p.Sh * p.W + wsx * p.Sw;
    }
    uint16_t v[8][2];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const bool cok = c0 + wid + 8 * i < p.C;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        v[i][j] = 0;
        if (cok && pok[j]) v[i][j] = src[j][8 * i * HW];
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) pre_smem[(wid + 8 * i) * kPitch + j * 32 + lane] = v[i][j];
  }
  __syncthreads();
  // writes: a thread takes one pixel and 8 consecutive channels (16 bytes); 512 such pieces per tile
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const int piece = threadIdx.x + 256 * k;
    const int pl = piece >> 3, cg = piece & 7;
    const int64_t gp = g0 + pl;
    const int c = c0 + cg * 8;
    if (gp < p.total_pix && c < p.Cp) {
      uint32_t wd[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        wd[i] = static_cast<uint32_t>(pre_smem[(cg * 8 + 2 * i) * kPitch + pl]) |
                (static_cast<uint32_t>(pre_smem[(cg * 8 + 2 * i + 1) * kPitch + pl]) << 16);
      *reinterpret_cast<uint4*>(xs + gp * p.Cp + c) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
    }
  }
}

// Few input channels (Kw*Cp <= 64): "row window" layout.  The activations are copied to
// (N, Hp, Wpa, Cp) with the border cells written out as zeros.  In that copy the Kw*Cp values
// that one filter row meets at output column w' are contiguous and start Sw*Cp elements after
// those of w'-1, so a tensor map whose second dimension has that (overlapping) stride delivers,
// per filter row, a ready K-major tile of 64 values per output column.  The weights go to
// (O, Kh, 64) with zeros in the unused tail of every 64.
__global__ void __launch_bounds__(256) rowwin_pack_x(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                                     int channels_last, int C, int H, int W, int Hp, int Wpa, int Cp,
                                                     int ph, int pw) {
  // one block per padded row (n, hp); threads walk the row's pixels
  const int64_t rowid = blockIdx.x;
  const int hp = static_cast<int>(rowid % Hp);
  const int64_t n = rowid / Hp;
  const int h = hp - ph;
  const bool row_ok = h >= 0 && h < H;
  uint16_t* orow = out + rowid * Wpa * Cp;
  for (int wp = threadIdx.x; wp < Wpa; wp += blockDim.x) {
    const int w = wp - pw;
    const bool inside = row_ok && w >= 0 && w < W;
    for (int c0 = 0; c0 < Cp; c0 += 8) {
      union { uint4 v; uint16_t e[8]; } px;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = c0 + i;
        uint16_t val = 0;
        if (inside && c < C)
          val = channels_last ? in[((n * H + h) * W + w) * C + c] : in[((n * C + c) * H + h) * static_cast<int64_t>(W) + w];
        px.e[i] = val;
      }
      *reinterpret_cast<uint4*>(orow + static_cast<int64_t>(wp) * Cp + c0) = px.v;
    }
  }
}

__global__ void __launch_bounds__(256) rowwin_pack_w(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                                     int channels_last, int64_t O, int64_t C, int64_t Kh, int64_t Kw,
                                                     int Cp) {
  const int64_t total = O * Kh * 64;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int j = static_cast<int>(e % 64);
    const int64_t kh = (e / 64) % Kh, o = e / (64 * Kh);
    const int kw = j / Cp, c = j % Cp;
    uint16_t val = 0;
    if (kw < Kw && c < C) val = channels_last ? in[((o * Kh + kh) * Kw + kw) * C + c] : in[((o * C + c) * Kh + kh) * Kw + kw];
    out[e] = val;
  }
}

// ------------------------------------------------------------------------
// tcgen05 / TMA building blocks (inline PTX)
// ------------------------------------------------------------------------

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // a wait that lasts 2 s has failed

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ uint64_t global_timer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the block is giving up: either this wait
// ran out of time (it then raises the block's abort flag and the device status
// word) or another role of the block already did.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    __nanosleep(40);
    if ((++spins & 0xFFu) == 0) {
      if (*abort_flag) return false;
      if (global_timer() - t0 > limit_ns) {
        *abort_flag = 1;
        atomicOr(&g_status, 1u);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
// im2col-mode load of a (pixels x channels) box: coordinates are the first
// window origin (c, w, h, n); the filter offset (kw, kh) is added by the TMA unit.
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                uint16_t kw, uint16_t kh, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(kw), "h"(kh)
      : "memory");
}

// Prefetches into L2 with the coordinates of a later load.  A kernel launched with programmatic stream
// serialisation issues them BEFORE it waits for its predecessor: a prefetch consumes nothing, and L2 is where all
// SMs' writes meet, so a line the predecessor still writes afterwards is simply updated there.  The operands of
// the first tiles then come from L2 instead of from DRAM once the wait is over.
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* map, int c, int w, int h, int n) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n) : "memory");
}
__device__ __forceinline__ void tma_prefetch_im2col(const CUtensorMap* map, int c, int w, int h, int n, uint16_t kw, uint16_t kh) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.im2col [%0, {%1, %2, %3, %4}], {%5, %6};"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "h"(kw), "h"(kh) : "memory");
}

// ---- two-block clusters (CTA pairs): one tcgen05.mma spans the tensor cores and the shared
// memory of both blocks of a pair; barriers that both blocks feed live in the pair's first block.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `saddr` (a shared::cta address of this block) in block `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Pair forms of the loads: the data lands in this block, the bytes are counted on a barrier that
// may sit in the other block of the pair (`bar` is a shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col_pair(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                     uint16_t kw, uint16_t kh, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(kw), "h"(kh)
      : "memory");
}

// One lane of the (converged) warp.  The MMA warps run their loops warp-uniformly and predicate only the
// tcgen05 instructions on this lane: descriptors and barrier addresses then stay warp-uniform values.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.b32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, M = 128, N from the instruction descriptor, K = 16.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Pair forms: issued by one thread of the pair's first block; the commit arrives at the barrier
// at the same offset in both blocks.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(static_cast<uint16_t>(3))
      : "memory");
}
// D (256 rows: 128 TMEM lanes in each block) (+)= A (128 rows from each block) * B^T (N/2 rows from each block)
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_load_32cols(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile.
//   bits  0-13 start address >> 4      bits 16-29 leading byte offset >> 4
//   bits 32-45 stride byte offset >> 4 bits 46-47 descriptor version (1)
//   bits 61-63 swizzle: 0 none, 2 128-byte
// 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart (SBO).
// No swizzle: 8x16-byte core matrices; LBO between cores along K, SBO along rows.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swz) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= static_cast<uint64_t>(swz) << 61;
  return d;
}

// Instruction descriptor, kind::f16: D fp32 (bits 4-5 = 1), A and B bf16
// (bits 7-9, 10-12 = 1), both K-major (bits 15, 16 = 0), N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

// ------------------------------------------------------------------------
// The GEMM kernel
// ------------------------------------------------------------------------

constexpr int kBM = 128;
constexpr int kBK = 64;          // bf16 elements per K block = one 128-byte swizzle row
constexpr int kTcThreads = 224;  // warp 0 TMA (A), warp 1 MMA + TMEM, warps 2-5 epilogue, warp 6 TMA (B)

enum AMode { kDense = 0, kIm2col = 1, kIm2colGranule = 2, kRowWin = 3, kChwPix = 4 };

struct TcParams {
  int64_t M, O, K;        // K as laid out in B (for conv: Kh*Kw*Cp)
  int tiles_m, tiles_n, kblocks;
  int relu;
  int out_nchw;           // store (image, O, H'W') instead of [M,O]: squeeze + transpose (0 3 1 2) of Fig. 2a
  int tma_store;          // result rows are 16-byte multiples: the epilogue may use TMA stores
  int out_bf16;           // results rounded to bf16 and stored as 2-byte elements (never with a K split: the
                          // partial planes stay fp32 and the summing kernel rounds)
  // conv only
  int Cp, Kh, Kw, Sh, Sw, ph, pw, Ho, Wo;
  int cchunks;            // kIm2col: 64-channel chunks per tap; kIm2colGranule: 8-channel granules per tap
  FastDiv div_tiles_n, div_wo, div_howo;
  // K split (Section 5.4: a split of the contracted dimension turns dotProd into reduceSum over
  // partial dotProds): unit u = tile u / ksplit, K blocks [s*kper, (s+1)*kper), s = u % ksplit.
  // With ksplit > 1 the kernel writes partial [s][M][O] planes and a second kernel adds them up.
  int ksplit, kper;
  FastDiv div_ksplit;
  int prefetch;           // operands may be prefetched into L2 before the dependency wait (not when the call's own
                          // layout copies, the predecessor in the stream, are what writes them)
  // kRowWin only: one tile = (up to) 128 outputs of one output row
  int Hp, segs;           // padded input rows per image; 128-wide segments per output row
  FastDiv div_segs, div_ho;
  // Pairs only: tiles of two widths.  When the tile count is not a multiple of the resident pairs the last
  // wave is partly empty; replacing some BN-wide tiles by half-wide ones evens the pairs' loads out.  Row band
  // tm holds w(tm) = wA (tm < bA) or wA - 1 wide tiles from column 0 on, then half-wide tiles up to O.  Units
  // count the wide tiles of all bands first (n_wide of them), then the half-wide ones (nA per band for
  // tm < bA, nA + 2 per later band).
  int mix, n_wide, wA, bA, nA;
  // kChwPix only: 1x1 windows over (C,H,W) items read where they are.  A tile is two output rows of one image in
  // a pitch of 64 pixels: tensor-memory lane m = 64 * j + w is input pixel (row (2 * ti + j) * Sh, column w).
  // With unit strides the image is one run of H*W pixels instead (pix_flat): a tile is 128 consecutive pixels.
  int pix_tpi, pix_w;     // tiles per image = ceil(Ho / 2); input width (w >= pix_w: zero fill, dropped)
  int pix_flat, pix_hw;   // flat form: tiles per image = ceil(H*W / 128)
  FastDiv div_pix_tpi;
};

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n, uint32_t bar);

struct TileAt { int tm, n0, width; };

// Work unit (without the K-split index) -> row band, first column and width of its tile.
template <int BN>
__device__ __forceinline__ TileAt decode_tile(const TcParams& p, uint32_t t) {
  TileAt at;
  if (!p.mix) {
    uint32_t tm, tn;
    p.div_tiles_n.divmod(t, tm, tn);
    at.tm = static_cast<int>(tm); at.n0 = static_cast<int>(tn) * BN; at.width = BN;
    return at;
  }
  const int u = static_cast<int>(t);
  if (u < p.n_wide) {
    const int first = p.bA * p.wA;
    int j;
    if (u < first) { at.tm = u / p.wA; j = u - at.tm * p.wA; }
    else { const int v = u - first, w = p.wA - 1; at.tm = v / w; j = v - at.tm * w; at.tm += p.bA; }
    at.n0 = j * BN; at.width = BN;
    return at;
  }
  const int v = u - p.n_wide, first = p.bA * p.nA;
  int j;
  if (v < first) { at.tm = v / p.nA; j = v - at.tm * p.nA; at.n0 = p.wA * BN + j * (BN / 2); }
  else { const int x = v - first, n = p.nA + 2; at.tm = x / n; j = x - at.tm * n; at.tm += p.bA; at.n0 = (p.wA - 1) * BN + j * (BN / 2); }
  at.width = BN / 2;
  return at;
}

// A stage holds G K-blocks of 64 (G A sub-tiles, then G B sub-tiles) behind one pair of barriers.
// OCC = blocks per SM the configuration is sized for (2 only for BN <= 128: TMEM has 512 columns).
// CTAS = 2: two blocks on neighbouring SMs (a cluster) share one 256 x BN tile; each stages its own
// 128 rows of A and BN/2 rows of B, and one thread of the first block issues MMAs that span both.
template <int BN, int G, int OCC, int CTAS = 1>
struct TcCfg {
  static constexpr int kStageA = kBM * kBK * 2;
  static constexpr int kStageB = (BN / CTAS) * kBK * 2;
  static constexpr int kStage = G * (kStageA + kStageB);
  static constexpr int kEpiBufs = OCC == 2 ? 1 : 2;          // 32x32 fp32 staging tiles per epilogue warp
  static constexpr int kEpiBytes = 4 * kEpiBufs * 4096;
  static constexpr int kBudget = (OCC == 2 ? 113 * 1024 : 232448) - kEpiBytes - 1024 - 256;
  static constexpr int kStages = kBudget / kStage > 8 ? 8 : kBudget / kStage;
  static constexpr int kTmemCols = (2 * BN > 256) ? 512 : (2 * BN > 128 ? 256 : 128);   // power of two
  static constexpr int kSmemBytes = kStages * kStage + kEpiBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN, int MODE, int G, int OCC, int CTAS>
__global__ void __launch_bounds__(kTcThreads, OCC)
dot_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
       const __grid_constant__ CUtensorMap map_c, float* __restrict__ out, const TcParams p) {
  using Cfg = TcCfg<BN, G, OCC, CTAS>;
  static_assert(CTAS == 1 || (CTAS == 2 && (MODE == kDense || MODE == kIm2col)), "pairs: dense and im2col tiles only");
  static_assert(MODE != kChwPix || (CTAS == 1 && G == 1), "pixel-major A: one K block per stage, single blocks");
  static_assert(Cfg::kStages >= 2, "ring too shallow");
  extern __shared__ unsigned char smem_raw[];
  // operand tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  unsigned char* gen_tiles = smem_raw + (tiles - raw);
  const uint32_t epi_base = tiles + Cfg::kStages * Cfg::kStage;      // 1024-byte aligned staging tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_tiles + Cfg::kStages * Cfg::kStage + Cfg::kEpiBytes);
  const uint32_t bar_full = smem_u32(bars);                          // [kStages]
  const uint32_t bar_empty = bar_full + 8 * Cfg::kStages;            // [kStages]
  const uint32_t bar_tfull = bar_empty + 8 * Cfg::kStages;           // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * Cfg::kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // position in the pair: block 0 owns the barriers both blocks feed and issues the MMAs
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;
  // the tensor maps are kernel parameters: their fetch starts now, under the set-up
  if (threadIdx.x == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
    if (p.tma_store) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_c)) : "memory");
  }

  if (threadIdx.x == 0) {
    // full: the two producer threads of block 0 announce the bytes of the whole pair
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(bar_full + 8 * s, 2); mbar_init(bar_empty + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + 8 * a, 1); mbar_init(bar_tempty + 8 * a, 4 * CTAS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) {   // the same warp of both blocks allocates the same columns in both tensor memories
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(static_cast<uint32_t>(Cfg::kTmemCols))
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(static_cast<uint32_t>(Cfg::kTmemCols))
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // the other block's barriers exist before anything signals them
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // work units (p.tiles_m counts 128*CTAS-row tiles)
  const int num_tiles = p.mix ? p.n_wide + p.bA * p.nA + (p.tiles_m - p.bA) * (p.nA + 2) : p.tiles_m * p.tiles_n * p.ksplit;
  const int unit0 = static_cast<int>(blockIdx.x) / CTAS, unit_step = static_cast<int>(gridDim.x) / CTAS;
  // while the predecessor drains: the operands of this block's first unit (at most 4 K blocks of it) on their
  // way into L2
  if (p.prefetch && (MODE == kDense || MODE == kIm2col) && (warp == 0 || warp == 6) && unit0 < num_tiles) {
    if (elect_one()) {
      uint32_t t, ks;
      p.div_ksplit.divmod(static_cast<uint32_t>(unit0), t, ks);
      const TileAt at = decode_tile<BN>(p, t);
      const int kb_begin = static_cast<int>(ks) * p.kper, kb_end = min(min(p.kblocks, kb_begin + p.kper), kb_begin + 4);
      const int m0 = (at.tm * CTAS + static_cast<int>(rank)) * kBM;
      const int n0 = at.n0 + static_cast<int>(rank) * (at.width / CTAS);
      constexpr int kBoxesB = CTAS == 2 ? 2 : 1;   // pairs: B boxes are BN/4 rows high
      if (MODE == kDense) {
        for (int kb = kb_begin; kb < kb_end; ++kb) {
          if (warp == 0) tma_prefetch_2d(&map_a, kb * kBK, m0);
          else
            for (int h = 0; h < kBoxesB; ++h) tma_prefetch_2d(&map_b, kb * kBK, n0 + h * (BN / 4));
        }
      } else {
        uint32_t im, rem, ho, wo;
        p.div_howo.divmod(static_cast<uint32_t>(m0), im, rem);
        p.div_wo.divmod(rem, ho, wo);
        const int tap0 = kb_begin / p.cchunks;
        int cc = kb_begin - tap0 * p.cchunks, kh = tap0 / p.Kw, kw = tap0 - kh * p.Kw;
        for (int kb = kb_begin; kb < kb_end; ++kb) {
          if (warp == 0)
            tma_prefetch_im2col(&map_a, cc * kBK, static_cast<int>(wo) * p.Sw - p.pw, static_cast<int>(ho) * p.Sh - p.ph,
                                static_cast<int>(im), static_cast<uint16_t>(kw), static_cast<uint16_t>(kh));
          else
            for (int h = 0; h < kBoxesB; ++h) tma_prefetch_2d(&map_b, (kh * p.Kw + kw) * p.Cp + cc * kBK, n0 + h * (BN / 4));
          if (++cc == p.cchunks) { cc = 0; if (++kw == p.Kw) { kw = 0; ++kh; } }
        }
      }
    }
  }
  pdl_wait();
  pdl_launch_dependents();


  if (warp == 0 || warp == 6) {
    // ---------------- TMA producers: warp 0 stages A, warp 6 stages B ----------------
    // The whole warp runs the loop (warp-uniform control flow and values); one elected lane issues the
    // copies.  Issued from inside a one-lane branch, every TMA or MMA instruction cost its thread 60-150
    // cycles of operand shuffling; from uniform code it costs 15-30.
    const bool load_a = warp == 0;
    const bool leader = elect_one();
    {
      uint32_t s = 0, ph = 0;   // ring slot and its phase, advanced by hand (no division in this loop)
      bool ok = true;
      for (int u = unit0; u < num_tiles && ok; u += unit_step) {
        uint32_t t, ks;
        p.div_ksplit.divmod(static_cast<uint32_t>(u), t, ks);
        const TileAt at = decode_tile<BN>(p, t);
        const uint32_t tm = static_cast<uint32_t>(at.tm);
        const int kb_begin = static_cast<int>(ks) * p.kper, kb_end = min(p.kblocks, kb_begin + p.kper);
        // this block's 128 rows of A and its share of the tile's rows of B (pairs fetch B in boxes of BN/4 rows:
        // two per K block for a full-width tile, one for a half-width tile)
        const int m0 = (at.tm * CTAS + static_cast<int>(rank)) * kBM;
        const int n0 = at.n0 + static_cast<int>(rank) * (at.width / CTAS);
        const int b_bytes = CTAS == 2 ? (at.width == BN ? Cfg::kStageB : Cfg::kStageB / 2) : Cfg::kStageB;
        int wbase = 0, hbase = 0, img = 0;
        if (MODE == kRowWin) {
          if (load_a) {   // tile -> (output row, segment) -> first padded input row
            uint32_t row, seg, im, ho;
            p.div_segs.divmod(tm, row, seg);
            p.div_ho.divmod(row, im, ho);
            wbase = static_cast<int>(seg) * kBM;
            hbase = static_cast<int>(im) * p.Hp + static_cast<int>(ho) * p.Sh;
          }
        } else if (MODE == kChwPix) {
          if (load_a) {   // tile -> (image, pair of output rows)
            uint32_t im, ti;
            p.div_pix_tpi.divmod(tm, im, ti);
            img = static_cast<int>(im);
            hbase = static_cast<int>(ti) * 2;
          }
        } else if (MODE != kDense && load_a) {
          uint32_t im, rem, ho, wo;
          p.div_howo.divmod(static_cast<uint32_t>(m0), im, rem);
          p.div_wo.divmod(rem, ho, wo);
          img = static_cast<int>(im);
          wbase = static_cast<int>(wo) * p.Sw - p.pw;
          hbase = static_cast<int>(ho) * p.Sh - p.ph;
        }
        // filter position of the next K block, advanced without divisions
        int cc = 0, kw = 0, kh = 0;
        if (MODE == kIm2col && kb_begin > 0) {
          const int tap = kb_begin / p.cchunks;
          cc = kb_begin - tap * p.cchunks;
          kh = tap / p.Kw;
          kw = tap - kh * p.Kw;
        }
        for (int kb0 = kb_begin; kb0 < kb_end; kb0 += G) {
          if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t full = CTAS == 2 ? map_to_cta(bar_full + 8 * s, 0) : bar_full + 8 * s;
          const uint32_t stage = tiles + s * Cfg::kStage;
          const int nsub = min(G, kb_end - kb0);
          if (rank == 0 && leader) mbar_expect_tx(bar_full + 8 * s, nsub * CTAS * (load_a ? Cfg::kStageA : b_bytes));
#pragma unroll 1
          for (int j = 0; j < nsub; ++j) {
            const int kb = kb0 + j;
            if (leader) {
            const uint32_t sa = stage + j * Cfg::kStageA, sb = stage + G * Cfg::kStageA + j * Cfg::kStageB;
            if (CTAS == 2) {
              if (MODE == kDense) {
                if (load_a) tma_load_2d_pair(sa, &map_a, kb * kBK, m0, full);
                else {
                  tma_load_2d_pair(sb, &map_b, kb * kBK, n0, full);
                  if (at.width == BN) tma_load_2d_pair(sb + Cfg::kStageB / 2, &map_b, kb * kBK, n0 + BN / 4, full);
                }
              } else {
                if (load_a)
                  tma_load_im2col_pair(sa, &map_a, cc * kBK, wbase, hbase, img, static_cast<uint16_t>(kw),
                                       static_cast<uint16_t>(kh), full);
                else {
                  const int kx = (kh * p.Kw + kw) * p.Cp + cc * kBK;
                  tma_load_2d_pair(sb, &map_b, kx, n0, full);
                  if (at.width == BN) tma_load_2d_pair(sb + Cfg::kStageB / 2, &map_b, kx, n0 + BN / 4, full);
                }
              }
            } else if (MODE == kDense) {
              if (load_a) tma_load_2d(sa, &map_a, kb * kBK, m0, full);
              else tma_load_2d(sb, &map_b, kb * kBK, n0, full);
            } else if (MODE == kRowWin) {
              // K block kb = filter row kb: 128 output columns x 64 values of padded input row hbase + kb
              if (load_a) tma_load_3d(sa, &map_a, 0, wbase, hbase + kb, full);
              else tma_load_2d(sb, &map_b, kb * kBK, n0, full);
            } else if (MODE == kChwPix) {
              // A arrives pixel-major: a box is 64 channels x one input row of 64 pixels (128 bytes per channel),
              // the tile's two rows 8 KB apart; pixels past the row's end read as zeros
              if (load_a) {
                if (p.pix_flat) {   // hbase = 2 * tile index: 64-pixel pieces hbase and hbase + 1 of the image
                  tma_load_3d(sa, &map_a, hbase * 64, kb * kBK, img, full);
                  tma_load_3d(sa + Cfg::kStageA / 2, &map_a, (hbase + 1) * 64, kb * kBK, img, full);
                } else {
                  tma_load_4d(sa, &map_a, 0, hbase * p.Sh, kb * kBK, img, full);
                  tma_load_4d(sa + Cfg::kStageA / 2, &map_a, 0, (hbase + 1) * p.Sh, kb * kBK, img, full);
                }
              } else {
                tma_load_2d(sb, &map_b, kb * kBK, n0, full);
              }
            } else if (MODE == kIm2col) {
              if (load_a)
                tma_load_im2col(sa, &map_a, cc * kBK, wbase, hbase, img, static_cast<uint16_t>(kw),
                                static_cast<uint16_t>(kh), full);
              else
                tma_load_2d(sb, &map_b, (kh * p.Kw + kw) * p.Cp + cc * kBK, n0, full);
            } else if (load_a) {
              // eight 8-channel granules per K block, each its own (pixels x 16 bytes) box
              const int taps = p.Kh * p.Kw;
#pragma unroll 1
              for (int g = 0; g < 8; ++g) {
                const int gi = kb * 8 + g;
                const int tap = gi / p.cchunks;
                // beyond the last tap: a box that lies outside the channel range reads as zeros
                const int c0 = tap < taps ? (gi % p.cchunks) * 8 : p.Cp;
                const int tp = tap < taps ? tap : 0;
                tma_load_im2col(sa + g * (kBM * 16), &map_a, c0, wbase, hbase, img, static_cast<uint16_t>(tp % p.Kw),
                                static_cast<uint16_t>(tp / p.Kw), full);
              }
            } else {
              tma_load_3d(sb, &map_b, 0, n0, kb * 8, full);
            }
            }
            // filter position of the next K block
            if (MODE == kIm2col) { if (++cc == p.cchunks) { cc = 0; if (++kw == p.Kw) { kw = 0; ++kh; } } }
          }
          if (++s == Cfg::kStages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (rank == 0) {
      const bool leader = elect_one();   // the loop is warp-uniform; this lane issues the MMAs and commits
      // (pixel-major A: bit 15 of the instruction descriptor = A is MN-major)
      constexpr uint32_t idesc_wide = make_idesc(kBM * CTAS, BN) | (MODE == kChwPix ? (1u << 15) : 0u),
                         idesc_half = make_idesc(kBM * CTAS, BN / 2);
      // MN-major A with the 128-byte swizzle: 64 pixels of one channel per 128-byte row, 8 channels per 1024-byte
      // group (SBO), the next 64 pixels LBO bytes further on
      const uint64_t desc_a0 = (MODE == kIm2colGranule) ? make_desc(tiles, kBM * 16, 128, 0)
                               : (MODE == kChwPix)      ? make_desc(tiles, Cfg::kStageA / 2, 1024, 2)
                                                        : make_desc(tiles, 16, 1024, 2);
      const uint64_t desc_b0 = (MODE == kIm2colGranule) ? make_desc(tiles + G * Cfg::kStageA, BN * 16, 128, 0)
                                                        : make_desc(tiles + G * Cfg::kStageA, 16, 1024, 2);
      uint32_t s = 0, ph = 0, tile_it = 0;
      bool ok = true;
      for (int u = unit0; u < num_tiles && ok; u += unit_step, ++tile_it) {
        const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
        uint32_t t, ks;
        p.div_ksplit.divmod(static_cast<uint32_t>(u), t, ks);
        const uint32_t idesc = (CTAS == 2 && p.mix && static_cast<int>(t) >= p.n_wide) ? idesc_half : idesc_wide;
        const int kb_begin = static_cast<int>(ks) * p.kper, kb_end = min(p.kblocks, kb_begin + p.kper);
        if (!mbar_wait(bar_tempty + 8 * acc, aph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb0 = kb_begin; kb0 < kb_end; kb0 += G) {
          if (!mbar_wait(bar_full + 8 * s, ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          // descriptors differ only in their start-address field (16-byte units): add offsets to a base
          const uint64_t da0 = desc_a0 + ((s * Cfg::kStage) >> 4);
          const uint64_t db0 = desc_b0 + ((s * Cfg::kStage) >> 4);
          const int nsub = min(G, kb_end - kb0);
#pragma unroll
          for (int j = 0; j < G; ++j) {
            if (j < nsub) {
#pragma unroll
              for (int k = 0; k < kBK / 16; ++k) {
                constexpr int kStepA = (MODE == kIm2colGranule) ? 2 * (kBM * 16) : (MODE == kChwPix ? 16 * 128 : 32);
                constexpr int kStepB = (MODE == kIm2colGranule) ? 2 * (BN * 16) : 32;
                const uint64_t da = da0 + ((j * Cfg::kStageA + k * kStepA) >> 4);
                const uint64_t db = db0 + ((j * Cfg::kStageB + k * kStepB) >> 4);
                const uint32_t accumulate = ((kb0 - kb_begin) | j | k) != 0 ? 1u : 0u;
                if (leader) {
                  if (CTAS == 2) tc_mma_bf16_pair(d_tmem, da, db, idesc, accumulate);
                  else tc_mma_bf16(d_tmem, da, db, idesc, accumulate);
                }
              }
            }
          }
          // one commit per stage (it costs the issuing thread a few hundred cycles): frees the
          // stage once these MMAs have read it
          if (leader) {
            if (CTAS == 2) tc_commit_pair(bar_empty + 8 * s);
            else tc_commit(bar_empty + 8 * s);
          }
          if (++s == Cfg::kStages) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) {
          if (CTAS == 2) tc_commit_pair(bar_tfull + 8 * acc);
          else tc_commit(bar_tfull + 8 * acc);
        }
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> (shared memory -> TMA store | global) ----------------
    const int q = warp & 3;   // TMEM lane quarter this warp may read
    const bool leader = elect_one();   // issues this warp's TMA stores (always the same lane: it owns the bulk groups)
    uint32_t tile_it = 0, chunk_it = 0;
    bool ok = true;
    const bool vec_ok = (p.O & 3) == 0;
    const uint32_t stage_buf = epi_base + q * (Cfg::kEpiBufs * 4096);   // this warp's 32 rows x 128 bytes tiles
    for (int u = unit0; u < num_tiles && ok; u += unit_step, ++tile_it) {
      const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
      uint32_t t, ks;
      p.div_ksplit.divmod(static_cast<uint32_t>(u), t, ks);
      const TileAt at = decode_tile<BN>(p, t);
      uint32_t tmu = static_cast<uint32_t>(at.tm);
      if (CTAS == 2) tmu = tmu * CTAS + rank;   // this block's 128 rows of the pair's tile
      const int tm = static_cast<int>(tmu);
      if (!mbar_wait(bar_tfull + 8 * acc, aph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      int64_t m = static_cast<int64_t>(tm) * kBM + q * 32 + lane;
      bool m_ok = m < p.M;
      uint32_t orow = 0, oseg = 0;
      if (MODE == kRowWin) {
        p.div_segs.divmod(tmu, orow, oseg);
        const int wloc = static_cast<int>(oseg) * kBM + q * 32 + lane;
        m = static_cast<int64_t>(orow) * p.Wo + wloc;
        m_ok = wloc < p.Wo;
      }
      if (MODE == kChwPix) {
        uint32_t im, ti;
        p.div_pix_tpi.divmod(tmu, im, ti);
        const int mloc = q * 32 + lane, w = mloc & 63, hh = static_cast<int>(ti) * 2 + (mloc >> 6);
        const int ow = w >> (p.Sw - 1);   // Sw is 1 or 2
        m = (static_cast<int64_t>(im) * p.Ho + hh) * p.Wo + ow;
        m_ok = hh < p.Ho && w < p.pix_w && (w & (p.Sw - 1)) == 0 && ow < p.Wo;
        if (p.pix_flat) {
          const int pixel = static_cast<int>(ti) * kBM + mloc;
          m = static_cast<int64_t>(im) * p.pix_hw + pixel;
          m_ok = pixel < p.pix_hw;
        }
      }
      const int64_t row_at = (static_cast<int64_t>(ks) * p.M + m) * p.O;   // partial plane ks (0 without a K split)
      float* row = out + row_at;
      int64_t col_at = 0;    // out_nchw: index of out[image][0][pixel]; channel o then lies o*H'W' further
      if (p.out_nchw && m_ok) {
        uint32_t img_o, pix_o;
        p.div_howo.divmod(static_cast<uint32_t>(m), img_o, pix_o);
        col_at = static_cast<int64_t>(img_o) * p.O * p.div_howo.d + pix_o;
      }
      float* col = out + col_at;
      // bf16 results through TMA stores go 64 columns at a time (128 bytes per row, as 32 fp32 columns do)
      const int cstep = (p.out_bf16 && p.tma_store) ? 64 : 32;
#pragma unroll 1
      for (int c = 0; c < at.width; c += cstep) {
        const int64_t n0 = static_cast<int64_t>(at.n0) + c;
        if (n0 >= p.O) break;   // uniform across the warp
        uint32_t r[32];
        tc_load_32cols(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + c, r);
        if (p.relu) {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(fmaxf(__uint_as_float(r[i]), 0.f));
        }
        if (cstep == 64) {
          // pack the first 32 columns, then fetch and pack the next 32: r[0..31] = 64 bf16 values of this row
#pragma unroll
          for (int i = 0; i < 16; ++i) r[i] = pack_bf16x2(r[2 * i], r[2 * i + 1]);
          uint32_t r2[32];
          tc_load_32cols(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + c + 32, r2);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            uint32_t a = r2[2 * i], b = r2[2 * i + 1];
            if (p.relu) { a = __float_as_uint(fmaxf(__uint_as_float(a), 0.f)); b = __float_as_uint(fmaxf(__uint_as_float(b), 0.f)); }
            r[16 + i] = pack_bf16x2(a, b);
          }
        }
        if (p.out_nchw) {
          // lanes hold consecutive pixels: for every channel the warp writes one contiguous run
          if (m_ok) {
            const int64_t plane = p.div_howo.d;
            if (p.out_bf16) {
              uint16_t* col16 = reinterpret_cast<uint16_t*>(out) + col_at;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n0 + i < p.O) col16[(n0 + i) * plane] = f32_to_bf16(__uint_as_float(r[i]));
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (n0 + i < p.O) col[(n0 + i) * plane] = __uint_as_float(r[i]);
            }
          }
        } else if (p.tma_store) {
          // 32x32 fp32 block: each lane parks its row in shared memory (16-byte pieces XOR-swizzled by
          // row, the 128-byte swizzle of the tensor map), then one lane hands the block to the TMA unit,
          // which writes whole 128-byte rows and clips at the matrix edge.
          const uint32_t buf = stage_buf + (Cfg::kEpiBufs == 2 ? (chunk_it & 1u) * 4096 : 0u);
          if (leader) {   // the store that last used this buffer has read it
            if (Cfg::kEpiBufs == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          }
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lane * 128 + ((j ^ (lane & 7)) << 4)),
                         "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3])
                         : "memory");
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (leader) {
            if (MODE == kRowWin)   // result viewed as (N*Ho, Wo, O): columns past Wo are clipped
              asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(
                               reinterpret_cast<uint64_t>(&map_c)),
                           "r"(static_cast<int>(n0)), "r"(static_cast<int>(oseg) * kBM + q * 32),
                           "r"(static_cast<int>(orow)), "r"(buf)
                           : "memory");
            else if (CTAS == 1 || tm * kBM + q * 32 < p.M)   // (planes, M, O): plane = K-split index, 0 without a split
              asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(
                               reinterpret_cast<uint64_t>(&map_c)),
                           "r"(static_cast<int>(n0)), "r"(tm * kBM + q * 32), "r"(static_cast<int>(ks)), "r"(buf)
                           : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          ++chunk_it;
        } else if (m_ok) {
          if (p.out_bf16) {
            uint16_t* row16 = reinterpret_cast<uint16_t*>(out) + row_at;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n0 + i < p.O) row16[n0 + i] = f32_to_bf16(__uint_as_float(r[i]));
          } else if (vec_ok && n0 + 32 <= p.O) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<uint4*>(row + n0 + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (n0 + i < p.O) row[n0 + i] = __uint_as_float(r[i]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2) mbar_arrive_cluster(map_to_cta(bar_tempty + 8 * acc, 0));
        else mbar_arrive(bar_tempty + 8 * acc);
      }
    }
    if (p.tma_store && leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // teardown: a block that gave up lets its copies in flight land before it leaves
  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_timer();
    while (global_timer() - t0 < 20000000ull) { }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // neither block leaves while the other may still signal it or read its tiles
  else __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(static_cast<uint32_t>(Cfg::kTmemCols))
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(static_cast<uint32_t>(Cfg::kTmemCols))
                   : "memory");
  }
}

// ------------------------------------------------------------------------
// Stride-1 convolutions with the input window tile resident in shared memory
// ------------------------------------------------------------------------
//
// windows (Section 4.2) of a stride-1 convolution overlap: neighbouring filter taps read the same
// input pixels one position apart.  With one 128-byte shared-memory row per pixel (64 channels),
// a tile of R output rows of one image needs the (R + Kh - 1) x Wb block of input pixels around it
// (Wb = W plus the horizontal padding), loaded ONCE by a tiled TMA box whose out-of-range cells
// read as zeros (the pad).  Number the tile's outputs m = oh * Wb + ow, i.e. in the pitch of the
// input block: the A operand of filter tap (kh, kw) is then the run of 128 shared-memory rows that
// starts kh * Wb + kw rows further down - the same bytes, another start address in the matrix
// descriptor (the 128-byte swizzle is a function of the shared-memory address, so a start on any
// row is consistent with what the TMA unit wrote).  Outputs with ow >= Wo are computed and dropped.
// Per tile the activations cross L2 -> SM once instead of Kh*Kw times.

constexpr int kHaloARows = 256;                     // shared-memory rows (pixels) per A stage
constexpr int kHaloAStage = kHaloARows * 128;
constexpr int kHaloMaxStages = 16;
constexpr int kHaloEpiBytes = 4 * 4096;             // one 32x32 fp32 staging tile per epilogue warp
constexpr int kHaloBarBytes = 640;
constexpr int kHaloSmemBudget = 232448 - 1024 - kHaloBarBytes - kHaloEpiBytes;

struct HaloParams {
  int64_t O;
  int relu;
  int out_bf16;   // results rounded to bf16 (O a multiple of 8)
  int N, Ho, Wo, Wb, R, tiles_m, tiles_n;   // tiles_m: M tiles, or pairs of them
  int Kh, Kw, Cp, cchunks;
  int tg, groups_per_chunk;                 // a B stage holds tg consecutive taps (a filter row, or one tap) of one chunk
  int ph, pw;
  int sa_stages, sb_stages, b_resident;     // b_resident: every B stage is loaded once per block and kept
  int prefetch;                             // operands may be prefetched into L2 before the dependency wait
  uint32_t a_bytes, b_bytes;                // bytes of one input box (64 channels); of one B stage
  FastDiv div_tiles_n, div_tpi, div_wb;     // tiles per image; padded width
};

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                 uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar)
      : "memory");
}

// BN: output channels per tile.  The weights are viewed as (64 channels, O, chunk, tap); one TMA box
// brings the BN x 64 slices of p.tg consecutive taps of one chunk.
// OCC = 2 (64-wide tiles): two blocks per SM, each with one input-box stage, so that one block's loads and
// epilogue run under the other's MMAs.
// CTAS = 2: two blocks on neighbouring SMs (a cluster) take two M tiles of the same column tile.  Each block
// stages the input box of its own tile and BN/2 rows of every weight box; one thread of the first block issues
// tcgen05.mma.cta_group::2 (M = 256), which reads both halves of the weights.  Per SM and MMA the shared
// memory then serves 4 KB of A and BN/2 rows of B instead of BN rows, and half the weight bytes cross L2 -> SM.
template <int BN, int OCC, int CTAS>
__global__ void __launch_bounds__(kTcThreads, OCC)
conv_halo(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
          float* __restrict__ out, const HaloParams p) {
  constexpr int kSubB = (BN / CTAS) * kBK * 2;       // one tap of B (this block's rows)
  constexpr int kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;
  const uint32_t kStageB = p.b_bytes;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - raw);
  const uint32_t a_base = base;
  const uint32_t b_base = a_base + p.sa_stages * kHaloAStage;
  const uint32_t epi_base = b_base + p.sb_stages * kStageB;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + (epi_base - base) + kHaloEpiBytes);
  const uint32_t bar_afull = smem_u32(bars);
  const uint32_t bar_aempty = bar_afull + 8 * kHaloMaxStages;
  const uint32_t bar_bfull = bar_aempty + 8 * kHaloMaxStages;
  const uint32_t bar_bempty = bar_bfull + 8 * kHaloMaxStages;
  const uint32_t bar_tfull = bar_bempty + 8 * kHaloMaxStages;
  const uint32_t bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4 * kHaloMaxStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  static_assert((4 * kHaloMaxStages + 4) * 8 + 8 <= kHaloBarBytes, "barrier block too small");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // position in the pair: block 0 owns the barriers both blocks feed and issues the MMAs
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;
  if (threadIdx.x == 32) {   // the tensor maps are kernel parameters: their fetch starts under the set-up
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
  }
  if (threadIdx.x == 0) {
    // full: one arrival, by the producer of block 0, which announces the bytes of the whole pair
    for (int s = 0; s < p.sa_stages; ++s) { mbar_init(bar_afull + 8 * s, 1); mbar_init(bar_aempty + 8 * s, 1); }
    for (int s = 0; s < p.sb_stages; ++s) { mbar_init(bar_bfull + 8 * s, 1); mbar_init(bar_bempty + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + 8 * a, 1); mbar_init(bar_tempty + 8 * a, 4 * CTAS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) {   // the same warp of both blocks allocates the same columns in both tensor memories
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(static_cast<uint32_t>(kTmemCols))
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(static_cast<uint32_t>(kTmemCols))
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // the other block's barriers exist before anything signals them
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // work units: p.tiles_m counts tiles of CTAS M tiles; this block takes M tile tm * CTAS + rank
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int unit0 = static_cast<int>(blockIdx.x) / CTAS, unit_step = static_cast<int>(gridDim.x) / CTAS;
  // while the predecessor drains: this block's input boxes, and one weight box per block, on their way into L2
  if (!p.prefetch) {
  } else if (warp == 0) {
    if (elect_one()) {
      for (int u = unit0; u < num_tiles; u += unit_step) {
        uint32_t tm, tn, img, ti;
        p.div_tiles_n.divmod(static_cast<uint32_t>(u), tm, tn);
        p.div_tpi.divmod(tm * CTAS + rank, img, ti);
        for (int cc = 0; cc < p.cchunks; ++cc)
          tma_prefetch_4d(&map_a, cc * kBK, -p.pw, static_cast<int>(ti) * p.R - p.ph, static_cast<int>(img));
      }
    }
  } else if (warp == 6) {
    if (elect_one()) {
      const int groups = p.cchunks * p.groups_per_chunk;
      for (int b = static_cast<int>(blockIdx.x); b < groups * p.tiles_n; b += static_cast<int>(gridDim.x)) {
        const int tn = b / groups, gi = b - tn * groups, cc = gi / p.groups_per_chunk, g = gi - cc * p.groups_per_chunk;
        for (int half = 0; half < CTAS; ++half)
          tma_prefetch_4d(&map_b, 0, tn * BN + half * (BN / CTAS), cc, g * p.tg);
      }
    }
  }
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    // ---------------- A producer: one input box per (tile, 64-channel chunk) ----------------
    // (warp-uniform loop, one elected lane issues: see dot_tc)
    const bool leader = elect_one();
    {
      uint32_t s = 0, ph = 0;
      bool ok = true;
      for (int u = unit0; u < num_tiles && ok; u += unit_step) {
        uint32_t tm, tn, img, ti;
        p.div_tiles_n.divmod(static_cast<uint32_t>(u), tm, tn);
        // an M tile past the last one (odd tile count) has img >= N: its box lies outside the tensor and reads as zeros
        p.div_tpi.divmod(tm * CTAS + rank, img, ti);
        const int h0 = static_cast<int>(ti) * p.R - p.ph;
        for (int cc = 0; cc < p.cchunks; ++cc) {
          if (!mbar_wait(bar_aempty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) {
            if (CTAS == 2) {
              if (rank == 0) mbar_expect_tx(bar_afull + 8 * s, 2 * p.a_bytes);
              tma_load_4d_pair(a_base + s * kHaloAStage, &map_a, cc * kBK, -p.pw, h0, static_cast<int>(img),
                               map_to_cta(bar_afull + 8 * s, 0));
            } else {
              mbar_expect_tx(bar_afull + 8 * s, p.a_bytes);
              tma_load_4d(a_base + s * kHaloAStage, &map_a, cc * kBK, -p.pw, h0, static_cast<int>(img), bar_afull + 8 * s);
            }
          }
          if (++s == static_cast<uint32_t>(p.sa_stages)) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 6) {
    // ---------------- B producer: stages in (chunk, tap group) order; once per block when resident ----------------
    const bool leader = elect_one();
    {
      uint32_t s = 0, ph = 0;
      bool ok = true;
      for (int u = unit0; u < num_tiles && ok; u += unit_step) {
        // this block's BN / CTAS rows of the column tile
        const int n0 = static_cast<int>(static_cast<uint32_t>(u) - p.div_tiles_n.div(static_cast<uint32_t>(u)) * p.tiles_n) * BN +
                       static_cast<int>(rank) * (BN / CTAS);
        for (int cc = 0; cc < p.cchunks && ok; ++cc) {
          for (int g = 0; g < p.groups_per_chunk; ++g) {
            if (!p.b_resident && !mbar_wait(bar_bempty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
            if (leader) {
              if (CTAS == 2) {
                if (rank == 0) mbar_expect_tx(bar_bfull + 8 * s, 2 * p.b_bytes);
                tma_load_4d_pair(b_base + s * kStageB, &map_b, 0, n0, cc, g * p.tg, map_to_cta(bar_bfull + 8 * s, 0));
              } else {
                mbar_expect_tx(bar_bfull + 8 * s, p.b_bytes);
                tma_load_4d(b_base + s * kStageB, &map_b, 0, n0, cc, g * p.tg, bar_bfull + 8 * s);
              }
            }
            if (++s == static_cast<uint32_t>(p.sb_stages)) { s = 0; ph ^= 1u; }
          }
        }
        if (p.b_resident) break;   // the weights stay where they are for every further tile
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    // One thread issues everything, so the loop is kept to the bare sequence: per chunk one wait for the
    // input box, per B stage one wait, p.tg * 4 MMAs whose descriptors advance by constants, one commit.
    if (rank == 0) {
      const bool leader = elect_one();
      constexpr uint32_t idesc = make_idesc(kBM * CTAS, BN);
      const uint64_t desc_a0 = make_desc(a_base, 16, 1024, 2);
      const uint64_t desc_b0 = make_desc(b_base, 16, 1024, 2);
      const uint32_t row_step = static_cast<uint32_t>(p.Wb * 128) >> 4;          // next filter row
      uint32_t sa = 0, pha = 0, sb = 0, phb = 0, tile_it = 0;
      bool ok = true;
      for (int u = unit0; u < num_tiles && ok; u += unit_step, ++tile_it) {
        const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
        if (!mbar_wait(bar_tempty + 8 * acc, aph ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t d_tmem = tmem_base + acc * BN;
        const bool wait_b = !p.b_resident || tile_it == 0;
        uint32_t accumulate = 0;
        for (int cc = 0; cc < p.cchunks && ok; ++cc) {
          if (!mbar_wait(bar_afull + 8 * sa, pha, abort_flag)) { ok = false; break; }
          // tap (kh, kw) reads the box from row kh * Wb + kw on: the group start advances by a filter
          // row (tg = Kw) or, with one tap per group, by one pixel with a jump at the end of a row
          uint64_t da_grp = desc_a0 + ((sa * static_cast<uint32_t>(kHaloAStage)) >> 4);
          int kw = 0;
          for (int g = 0; g < p.groups_per_chunk; ++g) {
            if (wait_b && !mbar_wait(bar_bfull + 8 * sb, phb, abort_flag)) { ok = false; break; }
            tc_fence_after();
            uint64_t da = da_grp, db = desc_b0 + ((sb * kStageB) >> 4);
#pragma unroll 1
            for (int t = 0; t < p.tg; ++t, da += 8, db += (kSubB >> 4)) {
              if (leader) {
              if (CTAS == 2) {
                tc_mma_bf16_pair(d_tmem, da, db, idesc, accumulate);
                tc_mma_bf16_pair(d_tmem, da + 2, db + 2, idesc, 1u);
                tc_mma_bf16_pair(d_tmem, da + 4, db + 4, idesc, 1u);
                tc_mma_bf16_pair(d_tmem, da + 6, db + 6, idesc, 1u);
              } else {
                tc_mma_bf16(d_tmem, da, db, idesc, accumulate);
                tc_mma_bf16(d_tmem, da + 2, db + 2, idesc, 1u);
                tc_mma_bf16(d_tmem, da + 4, db + 4, idesc, 1u);
                tc_mma_bf16(d_tmem, da + 6, db + 6, idesc, 1u);
              }
              }
              accumulate = 1u;
            }
            if (!p.b_resident && leader) { if (CTAS == 2) tc_commit_pair(bar_bempty + 8 * sb); else tc_commit(bar_bempty + 8 * sb); }
            if (++sb == static_cast<uint32_t>(p.sb_stages)) { sb = 0; phb ^= 1u; }
            if (p.tg == p.Kw) da_grp += row_step;
            else { da_grp += 8; if (++kw == p.Kw) { kw = 0; da_grp += row_step - 8u * p.Kw; } }
          }
          // the box may be overwritten once these MMAs retire
          if (leader) { if (CTAS == 2) tc_commit_pair(bar_aempty + 8 * sa); else tc_commit(bar_aempty + 8 * sa); }
          if (++sa == static_cast<uint32_t>(p.sa_stages)) { sa = 0; pha ^= 1u; }
        }
        if (ok && leader) { if (CTAS == 2) tc_commit_pair(bar_tfull + 8 * acc); else tc_commit(bar_tfull + 8 * acc); }
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> staged 32x32 blocks -> row-predicated global stores ----------------
    const int q = warp & 3;
    uint32_t tile_it = 0;
    bool ok = true;
    const uint32_t buf = epi_base + q * 4096;
    const int sub_row = lane >> 3, piece = lane & 7;
    for (int u = unit0; u < num_tiles && ok; u += unit_step, ++tile_it) {
      const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
      uint32_t tm, tn, img, ti;
      p.div_tiles_n.divmod(static_cast<uint32_t>(u), tm, tn);
      p.div_tpi.divmod(tm * CTAS + rank, img, ti);
      const bool tile_ok = static_cast<int>(img) < p.N;   // false for the filler tile of an odd tile count
      const int h0 = static_cast<int>(ti) * p.R;
      // the eight rows this lane stores (one per pass): offset of out[(img, h0 + oh, ow), 0], or -1 for a dropped row
      int64_t row_off[8];
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const uint32_t m = static_cast<uint32_t>(q * 32 + it * 4 + sub_row);
        uint32_t oh, ow;
        p.div_wb.divmod(m, oh, ow);
        const bool valid = tile_ok && static_cast<int>(oh) < p.R && h0 + static_cast<int>(oh) < p.Ho && static_cast<int>(ow) < p.Wo;
        row_off[it] = valid ? ((static_cast<int64_t>(img) * p.Ho + h0 + oh) * p.Wo + ow) * p.O : -1;
      }
      if (!mbar_wait(bar_tfull + 8 * acc, aph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int cstep = p.out_bf16 ? 64 : 32;   // a staged row is 128 bytes: 32 fp32 or 64 bf16 columns
#pragma unroll 1
      for (int c = 0; c < BN; c += cstep) {
        const int64_t n0 = static_cast<int64_t>(tn) * BN + c;
        if (n0 >= p.O) break;   // uniform across the warp
        uint32_t r[32];
        tc_load_32cols(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + c, r);
        if (p.relu) {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(fmaxf(__uint_as_float(r[i]), 0.f));
        }
        if (p.out_bf16) {
#pragma unroll
          for (int i = 0; i < 16; ++i) r[i] = pack_bf16x2(r[2 * i], r[2 * i + 1]);
          uint32_t r2[32];
          tc_load_32cols(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + c + 32, r2);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            uint32_t a = r2[2 * i], b = r2[2 * i + 1];
            if (p.relu) { a = __float_as_uint(fmaxf(__uint_as_float(a), 0.f)); b = __float_as_uint(fmaxf(__uint_as_float(b), 0.f)); }
            r[16 + i] = pack_bf16x2(a, b);
          }
        }
        __syncwarp();   // the previous block has been read back
#pragma unroll
        for (int j = 0; j < 8; ++j)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lane * 128 + ((j ^ (lane & 7)) << 4)),
                       "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3])
                       : "memory");
        __syncwarp();
        const int per_piece = p.out_bf16 ? 8 : 4;   // elements in 16 bytes; O is a multiple of it
        const bool col_ok = n0 + piece * per_piece < p.O;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int rr = it * 4 + sub_row;
          uint32_t v0, v1, v2, v3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3)
                       : "r"(buf + rr * 128 + ((piece ^ (rr & 7)) << 4))
                       : "memory");
          if (row_off[it] >= 0 && col_ok) {
            if (p.out_bf16)
              *reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(out) + row_off[it] + n0 + piece * 8) = make_uint4(v0, v1, v2, v3);
            else
              *reinterpret_cast<uint4*>(out + row_off[it] + n0 + piece * 4) = make_uint4(v0, v1, v2, v3);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2) mbar_arrive_cluster(map_to_cta(bar_tempty + 8 * acc, 0));
        else mbar_arrive(bar_tempty + 8 * acc);
      }
    }
  }

  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_timer();
    while (global_timer() - t0 < 20000000ull) { }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // neither block leaves while the other may still signal it or read its tiles
  else __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(static_cast<uint32_t>(kTmemCols))
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(static_cast<uint32_t>(kTmemCols))
                   : "memory");
  }
}

// ------------------------------------------------------------------------
// Few input channels: windows read in place from runs of the padded input rows
// ------------------------------------------------------------------------
//
// With pixels padded to Cp = 8 / Sw channels, the windows of neighbouring output columns start exactly
// 16 bytes apart in a (zero-bordered) row of the input, and a filter row of a window is Kw * Cp
// consecutive elements of that row.  The rows of the A operand are therefore overlapping pieces of one
// contiguous run of bytes.  The un-swizzled K-major operand layout of tcgen05.mma places row r of an
// 8-row group 16 bytes after row r-1 and K chunk j (8 elements) "leading byte offset" bytes after chunk
// j-1; with a leading byte offset of 16 and 128 bytes between 8-row groups the tensor core reads
//     A[r][k] = run[8 r + k]
// which is exactly windows(row, Kw*Cp, stride 8 elements) (Section 4.2) without forming it: shared memory
// holds each input row run ONCE (2 KB for 128 output columns), copied by one bulk copy per filter row, and
// cartProd/dotProd run over it as Kh * ceil(Kw*Cp/16) MMAs per tile.  The weights (a few KB) stay resident.

constexpr int kRunExpanders = 4;       // warp 0 copies raw rows, warps 6-9 widen them; warp 1 issues MMAs, warps 2-5 store results
constexpr int kRunThreads = 32 * (6 + kRunExpanders);
constexpr int kRunMaxStages = 4;
constexpr int kRunEpiBytes = 4 * 4096;   // one 32x32 fp32 staging tile per epilogue warp

struct RowRunParams {
  int64_t O;
  int relu;
  int out_bf16;   // results rounded to bf16 (O a multiple of 8)
  int out_nchw;   // results stored as (N, O, H', W'): squeeze + transpose (0 3 1 2) of Fig. 2a fused
  int C, H, W, Ho, Wo, Sh, Sw, Kh, Kw, ph, pw;
  int cp_log2;                  // pixels are widened to 8 / Sw = 2^cp_log2 channels
  int channels_last;            // items (H,W,C) / (Kh,Kw,C), else (C,H,W) / (C,Kh,Kw)
  int64_t xs_n, xs_h, xs_c;     // elements between images, rows and (for (C,H,W) items) channel planes
  int nseg;                     // raw copies per input row: 1 (pixels hold their channels) or C (one per plane)
  uint32_t raw_seg_bytes;       // shared-memory pitch of one raw copy, of the copies of a row, of a raw stage
  uint32_t raw_row_bytes, raw_stage_bytes;
  int raw_stages;
  int w_elems;                  // O * Kh * Kw * C (they fit the ring of row runs, where the block parks them once)
  int segs, tiles;              // 128-column segments per output row; tiles = N * Ho * segs
  // A block owns a strip of `strip` consecutive output rows of one image and segment.  Consecutive tiles share
  // Kh - Sh input rows, so the widened runs live in a ring of `ring` slots (input row hp of the strip at slot
  // (hp - first row) mod ring) and only the rows a tile adds - all Kh for the strip's first tile, min(Kh, Sh)
  // afterwards - are copied and widened.
  int strip, strips_per_img, ring;
  FastDiv div_spi, div_ring;
  int ksteps;                   // MMAs (K = 16) per filter row
  int bn;                       // MMA N: O rounded up to 16
  uint32_t seg_bytes;           // bytes of one run: 127 * 16 + ksteps * 32
  uint32_t slot_bytes;          // shared-memory pitch of a run
  uint32_t b_bytes;             // resident weights: Kh * ksteps * 2 chunks * bn rows * 16 bytes
  int stages;
  FastDiv div_segs, div_ho, div_nseg, div_bn;
};

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}
// The activations are read where they are, in either item layout.  Per tile (128 output columns of one output
// row) and filter row, the stretch of the input row that the tile's windows cover is brought into shared memory
// as it lies in global memory, by plain bulk copies of whole 16-byte pieces (one copy per row for (H,W,C) items,
// one per channel plane for (C,H,W) items); three warps then widen it into the padded row run: pixel wp of the
// run of filter row kh holds the C channels of input pixel (ho * Sh + kh - ph, seg * 128 * Sw + wp - pw), zeros
// for the border and for the channels past C.  A block walks down a strip of output rows, so every input row of the
// strip is copied and widened once and then serves the Kh / Sh tiles whose windows reach it.  The weights are
// rearranged into operand order by the whole block once, before the first tile.  Nothing passes through a
// global-memory copy.
// CT, CL: channel count and item layout as compile-time constants (CT = 0: both taken from p at run time).  The
// widening warps are bound by their instruction count per pixel; with constants it is a fifth of the general form.
template <int CT, int CL>
__global__ void __launch_bounds__(kRunThreads, 2)
conv_rowrun(const uint16_t* __restrict__ x, const uint16_t* __restrict__ wt,
            const __grid_constant__ CUtensorMap map_c, const RowRunParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - raw);
  const uint32_t epi_base = base;                                         // 1024-byte aligned staging tiles
  const uint32_t b_base = epi_base + kRunEpiBytes;
  const uint32_t a_base = b_base + ((p.b_bytes + 127u) & ~127u);
  const uint32_t r_base = a_base + static_cast<uint32_t>(p.ring) * p.slot_bytes;   // raw copies (slot_bytes is a multiple of 128)
  const uint32_t bars_off = (r_base - base) + static_cast<uint32_t>(p.raw_stages) * p.raw_stage_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + bars_off);
  const uint32_t bar_full = smem_u32(bars);                  // [kRunMaxStages] widened runs ready
  const uint32_t bar_empty = bar_full + 8 * kRunMaxStages;   // [kRunMaxStages] ... consumed by the MMAs
  const uint32_t bar_rfull = bar_empty + 8 * kRunMaxStages;  // [kRunMaxStages] raw copies landed
  const uint32_t bar_rempty = bar_rfull + 8 * kRunMaxStages; // [kRunMaxStages] ... widened
  const uint32_t bar_tfull = bar_rempty + 8 * kRunMaxStages; // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4 * kRunMaxStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t tmem_cols = 2 * p.bn <= 32 ? 32u : (2 * p.bn <= 64 ? 64u : (2 * p.bn <= 128 ? 128u : 256u));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 64) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_c)) : "memory");
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(bar_full + 8 * s, kRunExpanders); mbar_init(bar_empty + 8 * s, 1); }
    for (int s = 0; s < p.raw_stages; ++s) { mbar_init(bar_rfull + 8 * s, 1); mbar_init(bar_rempty + 8 * s, kRunExpanders); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + 8 * a, 1); mbar_init(bar_tempty + 8 * a, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int npx = static_cast<int>(p.seg_bytes >> (p.cp_log2 + 1));   // pixels of a run
  const int epx = p.channels_last ? p.C : 1;                          // elements per pixel in one raw copy
  // this block's strip: image, segment, first output row, number of tiles
  uint32_t strip_id, img_seg, img, seg;
  p.div_spi.divmod(blockIdx.x, img_seg, strip_id);
  p.div_segs.divmod(img_seg, img, seg);
  const int ho0 = static_cast<int>(strip_id) * p.strip;
  const int ntiles = min(p.strip, p.Ho - ho0);
  const int hp0 = ho0 * p.Sh;                       // first padded input row of the strip (row h = hp - ph)
  const int nnew_later = min(p.Kh, p.Sh);           // rows a tile adds (the first tile adds all Kh)
  const int w_first = static_cast<int>(seg) * (kBM * p.Sw) - p.pw;   // input column of run pixel 0
  const int w_lo = max(w_first, 0), w_hi = min(w_first + npx, p.W);
  // raw copies of tile t into raw stage r: lane i takes copy i = (new row, raw segment); called by warp 0.
  // With `only_prefetch` the same stretches are merely requested into L2 (before the dependency wait).
  auto copy_tile = [&](int t, uint32_t r, bool only_prefetch) {
    uint32_t j_l, c_l;
    p.div_nseg.divmod(static_cast<uint32_t>(lane), j_l, c_l);
    const int nnew = t == 0 ? p.Kh : nnew_later;
    const int h = hp0 + t * p.Sh + p.Kh - nnew + static_cast<int>(j_l) - p.ph;
    uint32_t size = 0;
    int64_t a0 = 0;
    if (static_cast<int>(j_l) < nnew && h >= 0 && h < p.H && w_hi > w_lo) {
      const int64_t e0 = static_cast<int64_t>(img) * p.xs_n + static_cast<int64_t>(h) * p.xs_h +
                         (p.channels_last ? static_cast<int64_t>(w_lo) * p.C : static_cast<int64_t>(c_l) * p.xs_c + w_lo);
      const int64_t b0 = e0 * 2, b1 = b0 + static_cast<int64_t>(w_hi - w_lo) * epx * 2;
      a0 = b0 & ~static_cast<int64_t>(15);                              // whole 16-byte pieces around the stretch;
      size = static_cast<uint32_t>(((b1 + 15) & ~static_cast<int64_t>(15)) - a0);   // the tensor's byte count is a multiple of 16
    }
    if (only_prefetch) {
      if (size)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<uint64_t>(x) + static_cast<uint64_t>(a0)),
                     "r"(size) : "memory");
      return;
    }
    const uint32_t total = __reduce_add_sync(0xffffffffu, size);
    if (lane == 0) mbar_expect_tx(bar_rfull + 8 * r, total);
    __syncwarp();
    if (size)
      bulk_copy_g2s(r_base + r * p.raw_stage_bytes + j_l * p.raw_row_bytes + c_l * p.raw_seg_bytes,
                    reinterpret_cast<const unsigned char*>(x) + a0, size, bar_rfull + 8 * r);
  };
  // while the predecessor drains: the rows of the first two tiles and the weights on their way into L2
  if (warp == 0) {
    for (int t = 0; t < min(ntiles, 2); ++t) copy_tile(t, 0, true);
  } else if (warp == 1) {
    const uint32_t wbytes = (static_cast<uint32_t>(p.w_elems) * 2u) & ~15u, piece = ((wbytes / 32u) + 15u) & ~15u;
    const uint32_t at = static_cast<uint32_t>(lane) * piece;
    if (piece && at < wbytes)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<uint64_t>(wt) + at),
                   "r"(min(piece, wbytes - at)) : "memory");
  }
  pdl_wait();
  pdl_launch_dependents();
  if (warp == 0 && ntiles > 0) copy_tile(0, 0, false);   // in flight while the block arranges the weights

  // ---- weights into operand order [kh][K chunk j][row o < bn][8 elements]: element kw * cp + c of filter row
  // kh sits at (j, i) = ((kw * cp + c) / 8, (kw * cp + c) % 8), zeros elsewhere.  The weight tensor is first
  // copied as it is (16-byte loads) into the ring of row runs, which nothing uses yet; every thread then
  // assembles 16-byte pieces (kh, j, o) from it.
  {
    uint16_t* wraw = reinterpret_cast<uint16_t*>(gen + (a_base - base));
    const int nvec = p.w_elems >> 3;
    for (int i = threadIdx.x; i < nvec; i += kRunThreads)
      reinterpret_cast<uint4*>(wraw)[i] = reinterpret_cast<const uint4*>(wt)[i];
    for (int i = nvec * 8 + threadIdx.x; i < p.w_elems; i += kRunThreads) wraw[i] = wt[i];
    __syncthreads();
    // a thread takes one (filter row, output channel) pair and writes its row of K: `chunks` pieces of 16 bytes
    const int chunks = 2 * p.ksteps, pairs = p.Kh * p.bn;
    const int cp_mask = (1 << p.cp_log2) - 1;
    uint4* wop = reinterpret_cast<uint4*>(gen + (b_base - base));
    // (H,W,C) items: element ((o Kh + kh) Kw + kw) C + c;  (C,H,W) items: ((o C + c) Kh + kh) Kw + kw
    // (with CT > 0 the channel count and the layout are constants and most of the index arithmetic folds)
    const int wC = CT > 0 ? CT : p.C;
    const bool wcl = CT > 0 ? CL != 0 : p.channels_last != 0;
    const int step_kw = wcl ? wC : 1, step_c = wcl ? 1 : p.Kh * p.Kw;
    for (int q = threadIdx.x; q < pairs; q += kRunThreads) {
      uint32_t kh, o;
      p.div_bn.divmod(static_cast<uint32_t>(q), kh, o);
      const bool row_ok = static_cast<int64_t>(o) < p.O;
      const int at = wcl ? static_cast<int>(o * p.Kh + kh) * p.Kw * wC : (static_cast<int>(o) * wC * p.Kh + static_cast<int>(kh)) * p.Kw;
      for (int j = 0; j < chunks; ++j) {
        uint32_t v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int el = j * 8 + i, kw = el >> p.cp_log2, c = el & cp_mask;
          v[i] = (row_ok && kw < p.Kw && c < wC) ? wraw[at + kw * step_kw + c * step_c] : 0u;
        }
        wop[(static_cast<int>(kh) * chunks + j) * p.bn + static_cast<int>(o)] =
            make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16), v[4] | (v[5] << 16), v[6] | (v[7] << 16));
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads them through the async proxy
    __syncthreads();
  }

  if (warp == 0) {
    // ---------------- raw copies: the first tile's went out before the weights were arranged ----------------
    uint32_t r = 1 % static_cast<uint32_t>(p.raw_stages), ph = p.raw_stages == 1 ? 1u : 0u;
    for (int t = 1; t < ntiles; ++t) {
      if (!mbar_wait(bar_rempty + 8 * r, ph ^ 1u, abort_flag)) break;
      copy_tile(t, r, false);
      if (++r == static_cast<uint32_t>(p.raw_stages)) { r = 0; ph ^= 1u; }
    }
  } else if (warp >= 6) {
    // ---------------- widening: raw rows -> padded row runs; the halves of the new rows dealt round robin to the warps ----------------
    const int eidx = warp - 6;
    const int cp = 1 << p.cp_log2;
    constexpr int kC = CT > 0 ? CT : 8;
    const int nch = CT > 0 ? CT : p.C;
    const bool cl = CT > 0 ? CL != 0 : p.channels_last != 0;
    const int epx_e = cl ? nch : 1;
    const int npx_half = ((npx >> 1) + 31) & ~31;
    uint32_t s = 0, ph = 0, r = 0, rph = 0;
    for (int t = 0; t < ntiles; ++t) {
      if (!mbar_wait(bar_rfull + 8 * r, rph, abort_flag)) break;
      if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag)) break;
      const int nnew = t == 0 ? p.Kh : nnew_later;
      const int hp_first = hp0 + t * p.Sh + p.Kh - nnew;
      for (int item = eidx; item < 2 * nnew; item += kRunExpanders) {
        const int j = item >> 1, half = item & 1;
        const int wp_begin = half ? npx_half : 0, wp_end = half ? npx : min(npx, npx_half);
        const int h = hp_first + j - p.ph;
        const bool row_ok = h >= 0 && h < p.H;
        // where the stretch starts inside its 16-byte aligned copy, per raw copy of this row
        const int64_t e0 = static_cast<int64_t>(img) * p.xs_n + static_cast<int64_t>(h) * p.xs_h +
                           (cl ? static_cast<int64_t>(w_lo) * nch : static_cast<int64_t>(w_lo));
        // element offset of the stretch inside its 16-byte aligned copy, per raw copy of this row
        uint32_t delta[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c)
          delta[c] = static_cast<uint32_t>((((e0 + (cl ? 0 : c * p.xs_c)) * 2) & 15) >> 1) +
                     (cl ? static_cast<uint32_t>(c) : static_cast<uint32_t>(c) * (p.raw_seg_bytes >> 1));
        uint32_t slot, lap;
        p.div_ring.divmod(static_cast<uint32_t>(hp_first + j - hp0), lap, slot);
        const uint16_t* src_row = reinterpret_cast<const uint16_t*>(gen + (r_base - base) + r * p.raw_stage_bytes +
                                                                    static_cast<uint32_t>(j) * p.raw_row_bytes);
        unsigned char* dst_row = gen + (a_base - base) + slot * p.slot_bytes;
        // four pixels per lane and trip: their loads are issued together
        for (int wp0 = wp_begin + lane; wp0 < wp_end; wp0 += 128) {
          uint32_t v[4][8];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int wp = wp0 + 32 * k, w = w_first + wp;
            const bool ok = row_ok && wp < wp_end && w >= w_lo && w < w_hi;
            const uint16_t* px = src_row + (ok ? (w - w_lo) * epx_e : 0);
#pragma unroll
            for (int c = 0; c < 8; ++c) v[k][c] = 0u;
#pragma unroll
            for (int c = 0; c < kC; ++c)
              if ((CT > 0 || c < nch) && ok) v[k][c] = px[delta[c]];
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int wp = wp0 + 32 * k;
            if (wp < wp_end) {
              unsigned char* dst = dst_row + (static_cast<uint32_t>(wp) << (p.cp_log2 + 1));
              const uint32_t w01 = v[k][0] | (v[k][1] << 16), w23 = v[k][2] | (v[k][3] << 16);
              if (cp == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(w01, w23, v[k][4] | (v[k][5] << 16), v[k][6] | (v[k][7] << 16));
              else if (cp == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(w01, w23);
              else if (cp == 2) *reinterpret_cast<uint32_t*>(dst) = w01;
              else *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(w01);
            }
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes before the tensor core's reads
      __syncwarp();
      if (lane == 0) { mbar_arrive(bar_full + 8 * s); mbar_arrive(bar_rempty + 8 * r); }
      if (++s == static_cast<uint32_t>(p.stages)) { s = 0; ph ^= 1u; }
      if (++r == static_cast<uint32_t>(p.raw_stages)) { r = 0; rph ^= 1u; }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    {
      const bool leader = elect_one();   // warp-uniform loop, one elected lane issues (see dot_tc)
      const uint32_t idesc = make_idesc(kBM, p.bn);
      const uint64_t desc_a0 = make_desc(a_base, 16, 128, 0);                                   // overlapping rows
      const uint64_t desc_b0 = make_desc(b_base, static_cast<uint32_t>(p.bn) * 16, 128, 0);    // [chunk][row][16 bytes]
      const uint32_t b_step = (2u * p.bn * 16u) >> 4;                                           // two K chunks per MMA
      uint32_t s = 0, ph = 0, tile_it = 0;
      bool ok = true;
      uint32_t slot = 0;   // ring slot of the tile's first input row: (t * Sh) mod ring
      const uint32_t slot_step = static_cast<uint32_t>(p.Sh) % static_cast<uint32_t>(p.ring);
      for (int t = 0; t < ntiles && ok; ++t, ++tile_it) {
        const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
        if (!mbar_wait(bar_tempty + 8 * acc, aph ^ 1u, abort_flag)) { ok = false; break; }
        if (!mbar_wait(bar_full + 8 * s, ph, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * p.bn;
        uint64_t db = desc_b0;
        uint32_t accumulate = 0, sl = slot;
        for (int kh = 0; kh < p.Kh; ++kh) {
          uint64_t da = desc_a0 + ((sl * p.slot_bytes) >> 4);
          if (++sl == static_cast<uint32_t>(p.ring)) sl = 0;
          for (int k = 0; k < p.ksteps; ++k, da += 2, db += b_step) {
            if (leader) tc_mma_bf16(d_tmem, da, db, idesc, accumulate);
            accumulate = 1u;
          }
        }
        if (leader) {
          tc_commit(bar_empty + 8 * s);
          tc_commit(bar_tfull + 8 * acc);
        }
        if (++s == static_cast<uint32_t>(p.stages)) { s = 0; ph ^= 1u; }
        slot += slot_step;
        if (slot >= static_cast<uint32_t>(p.ring)) slot -= p.ring;
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> swizzled 32x32 blocks -> TMA stores ----------------
    const int q = warp & 3;
    const bool leader = elect_one();   // issues this warp's TMA stores (always the same lane: it owns the bulk groups)
    uint32_t tile_it = 0, chunk_it = 0;
    bool ok = true;
    for (int t = 0; t < ntiles && ok; ++t, ++tile_it) {
      const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
      const uint32_t row = img * static_cast<uint32_t>(p.Ho) + static_cast<uint32_t>(ho0 + t);   // output row of the (N*Ho, Wo, O) view
      if (!mbar_wait(bar_tfull + 8 * acc, aph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int cstep = (p.out_bf16 && !p.out_nchw) ? 64 : 32;   // a staged row is 128 bytes: 32 fp32 or 64 bf16 columns
#pragma unroll 1
      for (int c = 0; c < p.bn; c += cstep) {
        if (c >= p.O) break;   // uniform across the warp
        uint32_t r[32];
        tc_load_32cols(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.bn + c, r);
        if (p.relu) {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(fmaxf(__uint_as_float(r[i]), 0.f));
        }
        if (p.out_nchw) {
          // squeeze + transpose fused: the 32 pixels x 32 channels block is parked channel-major (a lane writes
          // its pixel's value into every channel row: 32 lanes = one contiguous row piece, no bank conflict)
          // and leaves as one box {32 pixels, 1 row, 32 channels, 1 image} of the (W', H', O, N) view
          const uint32_t buf = epi_base + q * 4096;
          if (leader) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          __syncwarp();
          if (p.out_bf16) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              asm volatile("st.shared.b16 [%0], %1;" ::"r"(buf + i * 64 + lane * 2), "h"(f32_to_bf16(__uint_as_float(r[i]))) : "memory");
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              asm volatile("st.shared.b32 [%0], %1;" ::"r"(buf + i * 128 + lane * 4), "r"(r[i]) : "memory");
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (leader) {   // pixels past W' and channels past O are clipped
            asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(
                             reinterpret_cast<uint64_t>(&map_c)),
                         "r"(static_cast<int>(seg) * kBM + q * 32), "r"(ho0 + t), "r"(c), "r"(static_cast<int>(img)), "r"(buf)
                         : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          ++chunk_it;
          continue;
        }
        if (p.out_bf16) {
#pragma unroll
          for (int i = 0; i < 16; ++i) r[i] = pack_bf16x2(r[2 * i], r[2 * i + 1]);
          uint32_t r2[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) r2[i] = 0u;
          // the accumulator is bn columns wide: a second half exists only where c + 32 < bn
          if (c + 32 < p.bn) tc_load_32cols(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * p.bn + c + 32, r2);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            uint32_t a = r2[2 * i], b = r2[2 * i + 1];
            if (p.relu) { a = __float_as_uint(fmaxf(__uint_as_float(a), 0.f)); b = __float_as_uint(fmaxf(__uint_as_float(b), 0.f)); }
            r[16 + i] = pack_bf16x2(a, b);
          }
        }
        const uint32_t buf = epi_base + q * 4096;
        if (leader) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the previous store has read this buffer
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lane * 128 + ((j ^ (lane & 7)) << 4)),
                       "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3])
                       : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (leader) {   // result viewed as (N*Ho, Wo, O): columns past Wo and channels past O are clipped
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(
                           reinterpret_cast<uint64_t>(&map_c)),
                       "r"(c), "r"(static_cast<int>(seg) * kBM + q * 32), "r"(static_cast<int>(row)), "r"(buf)
                       : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        ++chunk_it;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
    }
    if (leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_timer();
    while (global_timer() - t0 < 20000000ull) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// One block waits on a barrier that nothing ever arrives at, with the same bounded wait the GEMM
// pipeline uses: it must give up after `limit_ns`, raise the status word and return normally.
__global__ void bounded_wait_selftest(uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_ns);
  __syncthreads();
}

// ------------------------------------------------------------------------
// Host side: tensor maps, dispatch
// ------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DriverApi {
  EncodeTiledFn tiled = nullptr;
  EncodeIm2colFn im2col = nullptr;
  bool ok = false;
};

const DriverApi& driver_api() {
  static DriverApi api;
  static std::once_flag once;
  std::call_once(once, [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || !f) return;
    api.tiled = reinterpret_cast<EncodeTiledFn>(f);
    f = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q) != cudaSuccess || !f) return;
    api.im2col = reinterpret_cast<EncodeIm2colFn>(f);
    api.ok = true;
  });
  return api;
}

// Encoded tensor maps, kept per argument list (base address, extents, strides, box, modes).  A program that
// calls the library on the same buffers again - every layer of a network on every step - skips the driver's
// encoding, which costs more host time than the rest of a call.  The map depends on nothing but its arguments,
// so a recycled address with the same geometry yields the same, still valid, map.
class TensorMapCache {
 public:
  template <typename Encode>
  bool get(const std::string& key, CUtensorMap* out, Encode&& encode) {
    {
      std::lock_guard<std::mutex> lock(mu_);
      auto it = maps_.find(key);
      if (it != maps_.end()) { *out = it->second; return true; }
    }
    if (!encode(out)) return false;
    std::lock_guard<std::mutex> lock(mu_);
    if (maps_.size() >= kMaxEntries) maps_.clear();
    maps_.emplace(key, *out);
    return true;
  }

 private:
  static constexpr size_t kMaxEntries = 4096;
  std::mutex mu_;
  std::unordered_map<std::string, CUtensorMap> maps_;
};

TensorMapCache& map_cache() {
  static TensorMapCache cache;
  return cache;
}

template <typename T>
void key_add(std::string* key, const T* v, size_t n) { key->append(reinterpret_cast<const char*>(v), n * sizeof(T)); }

bool encode_tiled_cached(CUtensorMap* m, CUtensorMapDataType dt, cuuint32_t rank, const void* base, const cuuint64_t* dims,
                         const cuuint64_t* strides, const cuuint32_t* box, const cuuint32_t* estr, CUtensorMapSwizzle swz,
                         CUtensorMapL2promotion l2) {
  std::string key;
  key.reserve(160);
  const uint32_t head[4] = {0u, static_cast<uint32_t>(dt), rank, static_cast<uint32_t>(swz) | (static_cast<uint32_t>(l2) << 8)};
  key_add(&key, head, 4);
  key_add(&key, &base, 1);
  key_add(&key, dims, rank);
  key_add(&key, strides, rank - 1);
  key_add(&key, box, rank);
  key_add(&key, estr, rank);
  return map_cache().get(key, m, [&](CUtensorMap* out) {
    return driver_api().tiled(out, dt, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                              l2, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  });
}

bool encode_im2col_cached(CUtensorMap* m, const void* base, const cuuint64_t* dims, const cuuint64_t* strides, const int* lower,
                          const int* upper, cuuint32_t channels, cuuint32_t pixels, const cuuint32_t* estr,
                          CUtensorMapSwizzle swz) {
  std::string key;
  key.reserve(160);
  const uint32_t head[4] = {1u, channels, pixels, static_cast<uint32_t>(swz)};
  key_add(&key, head, 4);
  key_add(&key, &base, 1);
  key_add(&key, dims, 4);
  key_add(&key, strides, 3);
  key_add(&key, lower, 2);
  key_add(&key, upper, 2);
  key_add(&key, estr, 4);
  return map_cache().get(key, m, [&](CUtensorMap* out) {
    return driver_api().im2col(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, lower, upper,
                               channels, pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  });
}

int num_sms() {
  static int sms[64] = {0};   // per device
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!sms[dev]) cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
  return sms[dev] > 0 ? sms[dev] : 148;
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// [rows, K] bf16 row-major, box {64, box_rows}, 128-byte swizzle, zero fill outside.
bool encode_kmajor_sw128(CUtensorMap* m, const void* base, int64_t rows, int64_t K, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {kBK, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// [rows, K] bf16 viewed as {8 elements, rows, K/8 granules}: one box {8, box_rows, 8}
// lands as [granule][row][16 bytes], the un-swizzled K-major core-matrix order.
bool encode_kmajor_granules(CUtensorMap* m, const void* base, int64_t rows, int64_t K, int box_rows) {
  const cuuint64_t dims[3] = {8, static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(K / 8)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(K) * 2, 16};
  const cuuint32_t box[3] = {8, static_cast<cuuint32_t>(box_rows), 8};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Channels-last activations (N,H,W,Cp) as an im2col tensor map: 128 window
// origins per box, `channels` channels per origin.
bool encode_im2col(CUtensorMap* m, const void* base, const DotProblem& d, int64_t Cp, int channels, bool swizzle) {
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(Cp), static_cast<cuuint64_t>(d.W), static_cast<cuuint64_t>(d.H),
                              static_cast<cuuint64_t>(d.N)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(Cp) * 2, static_cast<cuuint64_t>(d.W * Cp) * 2,
                                 static_cast<cuuint64_t>(d.H * d.W * Cp) * 2};
  const int lower[2] = {static_cast<int>(-d.pw_lo), static_cast<int>(-d.ph_lo)};
  const int upper[2] = {static_cast<int>(d.pw_hi - (d.Kw - 1)), static_cast<int>(d.ph_hi - (d.Kh - 1))};
  const cuuint32_t estr[4] = {1, static_cast<cuuint32_t>(d.Sw), static_cast<cuuint32_t>(d.Sh), 1};
  return encode_im2col_cached(m, base, dims, strides, lower, upper, static_cast<cuuint32_t>(channels), kBM, estr,
                              swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE);
}

// Result planes [planes, M, O]: boxes of 32 rows x 128 bytes (32 fp32 or 64 bf16 columns), 128-byte swizzle
// (what the epilogue stages).
bool encode_result(CUtensorMap* m, float* base, int64_t M, int64_t O, int64_t planes, bool bf16 = false) {
  const cuuint64_t es = bf16 ? 2 : 4;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(O), static_cast<cuuint64_t>(M), static_cast<cuuint64_t>(planes)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(O) * es, static_cast<cuuint64_t>(M * O) * es};
  const cuuint32_t box[3] = {bf16 ? 64u : 32u, 32, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode_tiled_cached(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// fp32 result of a row-window convolution viewed as (N*Ho, Wo, O): 32x32 boxes inside one output row.
bool encode_result_rows(CUtensorMap* m, float* base, int64_t rows, int64_t Wo, int64_t O, bool bf16 = false) {
  const cuuint64_t es = bf16 ? 2 : 4;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(O), static_cast<cuuint64_t>(Wo), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(O) * es, static_cast<cuuint64_t>(Wo * O) * es};
  const cuuint32_t box[3] = {bf16 ? 64u : 32u, 32, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode_tiled_cached(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// Result of the fused squeeze + transpose, (N, O, H', W') viewed as (W', H', O, N): boxes of 32 pixels of one
// output row x 32 channels, stored channel-major and un-swizzled.
bool encode_result_nchw(CUtensorMap* m, float* base, int64_t N, int64_t O, int64_t Ho, int64_t Wo, bool bf16) {
  const cuuint64_t es = bf16 ? 2 : 4;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(Wo), static_cast<cuuint64_t>(Ho), static_cast<cuuint64_t>(O),
                              static_cast<cuuint64_t>(N)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(Wo) * es, static_cast<cuuint64_t>(Ho * Wo) * es,
                                 static_cast<cuuint64_t>(O * Ho * Wo) * es};
  const cuuint32_t box[4] = {32, 1, 32, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return encode_tiled_cached(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// Row-window activations (N*Hp, Wpa, Cp): dimension 1 walks output columns with a stride of
// Sw*Cp elements, shorter than the 64 elements of dimension 0 (the windows overlap).
bool encode_rowwin(CUtensorMap* m, const void* base, int64_t rows, int64_t Wo, int64_t Wpa, int64_t Cp, int64_t Sw) {
  const cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(Wo), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(Sw * Cp) * 2, static_cast<cuuint64_t>(Wpa * Cp) * 2};
  const cuuint32_t box[3] = {64, kBM, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// The layout copies of a call (if it has any) are enqueued by this callable, which the launch functions run
// right before their own launch: everything that can fail without a launch - tensor-map encoding, function
// attributes, occupancy queries - has then been done, so a call refused for such a reason has enqueued nothing.
using PreLaunch = std::function<int()>;
inline int run_pre(const PreLaunch& pre) { return pre ? pre() : GL_OK; }

// Pairs: how many full-width tiles to keep so that, with units dealt out in turn (wide ones first), the most
// loaded pair has as little as possible.  Loads count half-width columns: a wide tile is 2, a half-wide tile 1.
// Sets p->mix and its fields when that beats all-wide tiles; returns the number of work units.
int plan_tile_mix(TcParams* p, int bn, int pairs) {
  const int bands = p->tiles_m, all_wide = bands * p->tiles_n;
  const int cu = static_cast<int>((p->O + bn / 2 - 1) / (bn / 2));   // half-wide columns per band
  if (pairs < 1 || cu < 2) return all_wide;
  const int old_span = 2 * ((all_wide + pairs - 1) / pairs);
  const int64_t units = static_cast<int64_t>(bands) * cu;
  const int span = static_cast<int>((units + pairs - 1) / pairs);
  const int wide = static_cast<int>(std::min<int64_t>(static_cast<int64_t>(pairs) * (span / 2), static_cast<int64_t>(bands) * (cu / 2)));
  const int64_t narrow = units - 2 * static_cast<int64_t>(wide);
  // dealing in turn: pair q gets wide tiles q, q + pairs, ...; the half-wide ones carry on from pair wide % pairs
  int worst = 0;
  for (int q = 0; q < pairs; ++q) {
    const int nw = wide / pairs + (q < wide % pairs ? 1 : 0);
    const int64_t first = ((q - wide % pairs) % pairs + pairs) % pairs;
    const int nn = narrow > first ? static_cast<int>((narrow - first + pairs - 1) / pairs) : 0;
    worst = std::max(worst, 2 * nw + nn);
  }
  if (worst >= old_span || wide < 1) return all_wide;
  p->mix = 1;
  p->n_wide = wide;
  p->wA = (wide + bands - 1) / bands;
  p->bA = wide - bands * (p->wA - 1);          // bands with wA wide tiles; the rest have wA - 1
  p->nA = cu - 2 * p->wA;
  return wide + static_cast<int>(narrow);
}

template <int BN, int MODE, int G, int OCC, int CTAS = 1>
int launch_tc(const CUtensorMap& ma, const CUtensorMap& mb, float* out, TcParams p, cudaStream_t st, const PreLaunch& pre) {
  using Cfg = TcCfg<BN, G, OCC, CTAS>;
  static bool attr_set_dev[64] = {false};   // per device; benign race: the attribute call is idempotent
  static int max_pairs_dev[64] = {0};       // CTAS == 2: pairs that can be resident at once
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return GL_ERR_CUDA;
  bool& attr_set = attr_set_dev[dev];
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute cluster_attr;
  std::memset(&cluster_attr, 0, sizeof(cluster_attr));
  cluster_attr.id = cudaLaunchAttributeClusterDimension;
  cluster_attr.val.clusterDim.x = CTAS;
  cluster_attr.val.clusterDim.y = 1;
  cluster_attr.val.clusterDim.z = 1;
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = st;
  cfg.attrs = &cluster_attr;
  cfg.numAttrs = CTAS == 2 ? 1 : 0;
  if (!attr_set) {
    if (cudaFuncSetAttribute(dot_tc<BN, MODE, G, OCC, CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes) != cudaSuccess)
      return GL_ERR_CUDA;
    if (CTAS == 2) {
      // a persistent grid must not exceed what is resident at once (SMs pair up within a GPC)
      cfg.gridDim = dim3(static_cast<unsigned>(num_sms() / 2 * 2));
      int pairs = 0;
      if (cudaOccupancyMaxActiveClusters(&pairs, dot_tc<BN, MODE, G, OCC, CTAS>, &cfg) != cudaSuccess || pairs < 1)
        return GL_ERR_CUDA;
      max_pairs_dev[dev] = pairs;
    }
    attr_set = true;
  }
  if (p.ksplit < 1) { p.ksplit = 1; p.kper = p.kblocks; }
  p.prefetch = pre ? 0 : 1;
  p.div_ksplit.set(p.ksplit);
  p.div_tiles_n.set(p.tiles_n);
  p.div_wo.set(p.Wo > 0 ? p.Wo : 1);
  p.div_howo.set(p.Wo > 0 ? static_cast<int64_t>(p.Wo) * p.Ho : 1);
  CUtensorMap mc;
  p.tma_store = (p.O % (p.out_bf16 ? 8 : 4) == 0 && !p.out_nchw && MODE != kChwPix) ? 1 : 0;
  if (MODE == kRowWin) {
    p.div_segs.set(p.segs);
    p.div_ho.set(p.Ho);
  }
  if (MODE == kChwPix) p.div_pix_tpi.set(p.pix_tpi);
  if (p.tma_store) {
    const bool ok = MODE == kRowWin ? encode_result_rows(&mc, out, p.M / p.Wo, p.Wo, p.O, p.out_bf16 != 0)
                                    : encode_result(&mc, out, p.M, p.O, p.ksplit, p.out_bf16 != 0);
    if (!ok) return GL_ERR_CUDA;
  } else {
    mc = ma;   // unused by the kernel; any valid map
  }
  int tiles = p.tiles_m * p.tiles_n * p.ksplit;
  p.mix = 0;
  if (CTAS == 2 && p.ksplit == 1) tiles = plan_tile_mix(&p, BN, std::min(max_pairs_dev[dev], num_sms() / 2));
  if (const int rc = run_pre(pre)) return rc;
  if (CTAS == 2) {
    const int pairs = std::min(tiles, std::min(max_pairs_dev[dev], num_sms() / 2));
    if (launch_pdl(dot_tc<BN, MODE, G, OCC, CTAS>, dim3(static_cast<unsigned>(2 * pairs)), dim3(kTcThreads),
                   Cfg::kSmemBytes, st, 2, ma, mb, mc, out, p) != cudaSuccess)
      return GL_ERR_CUDA;
    return GL_OK;
  }
  const int grid = tiles < OCC * num_sms() ? tiles : OCC * num_sms();
  return launch_pdl(dot_tc<BN, MODE, G, OCC, 1>, dim3(static_cast<unsigned>(grid)), dim3(kTcThreads), Cfg::kSmemBytes, st,
                    1, ma, mb, mc, out, p) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
}

// Wide tiles of a large problem are bound by operand traffic from L2 to the SMs; a pair of blocks
// sharing a 256x256 tile loads a third less per flop.  (The B tensor map then has boxes of bn/4 rows: two per
// block and K block for a full-width tile, one for a half-width tile.)
bool use_pair(int mode, int bn, const TcParams& p) {
  return bn == 256 && (mode == kDense || mode == kIm2col) && p.ksplit <= 1 && p.tiles_m >= 2;
}

template <int MODE>
int launch_tc_bn(int bn, const CUtensorMap& ma, const CUtensorMap& mb, float* out, const TcParams& p,
                 cudaStream_t st, const PreLaunch& pre) {
  switch (bn) {
    case 256:
      if (use_pair(MODE, bn, p)) {
        TcParams pp = p;
        pp.tiles_m = (p.tiles_m + 1) / 2;
        return launch_tc<256, (MODE == kDense || MODE == kIm2col) ? MODE : kDense, 1, 1, 2>(ma, mb, out, pp, st, pre);
      }
      return launch_tc<256, MODE, 1, 1>(ma, mb, out, p, st, pre);
    // narrower tiles are bound by the MMA-issuing thread (about 50 cycles per MMA, 250 per commit):
    // 128 wide: two K blocks per stage halve the commits; 64 wide: two blocks per SM interleave
    // their issue threads (measured on the 3x3 and 1x1 convolution shapes)
    case 128: return launch_tc<128, MODE, 2, 1>(ma, mb, out, p, st, pre);
    default:
      if (MODE == kIm2colGranule) return launch_tc<64, MODE, 1, 1>(ma, mb, out, p, st, pre);
      return launch_tc<64, MODE, 1, 2>(ma, mb, out, p, st, pre);
  }
}

// Column-tile width: 256 when that still leaves every SM a tile (wide tiles halve the operand
// traffic per flop), else the narrowest width that covers O in one or few tiles.
int pick_bn(int64_t M, int64_t O) {
  const int64_t tiles_m = (M + kBM - 1) / kBM;
  const int sms = num_sms();
  if (O > 128 && tiles_m * ((O + 255) / 256) >= sms) return 256;
  return O > 64 ? 128 : 64;
}

// compute reduceSum over the K-split partial planes (Section 5.4, last blocking rewrite), planes
// added in index order so that the result does not depend on scheduling; relu applied last.
__global__ void __launch_bounds__(256) splitk_reduce(const float* __restrict__ part, float* __restrict__ out,
                                                     int64_t n, int planes, int relu, int out_bf16) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t n4 = n >> 2;
  const float4* p4 = reinterpret_cast<const float4*>(part);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 acc = p4[i];
    for (int s = 1; s < planes; ++s) {
      const float4 v = p4[(s * n >> 2) + i];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (relu) { acc.x = fmaxf(acc.x, 0.f); acc.y = fmaxf(acc.y, 0.f); acc.z = fmaxf(acc.z, 0.f); acc.w = fmaxf(acc.w, 0.f); }
    if (out_bf16)
      reinterpret_cast<uint2*>(out)[i] = make_uint2(pack_bf16x2(__float_as_uint(acc.x), __float_as_uint(acc.y)),
                                                    pack_bf16x2(__float_as_uint(acc.z), __float_as_uint(acc.w)));
    else
      reinterpret_cast<float4*>(out)[i] = acc;
  }
}

// Tile width and K split for a [M,O] result with `kblocks` K blocks.  A problem with fewer tiles
// than a quarter of the SMs is split along K so that every SM gets a unit of at least four K blocks.
struct TilePlan { int bn = 64; int ksplit = 1; int kper = 0; size_t partial_bytes = 0; };

TilePlan plan_tiles(int64_t M, int64_t O, int64_t kblocks, bool may_split) {
  TilePlan tp;
  tp.bn = pick_bn(M, O);
  tp.kper = static_cast<int>(kblocks);
  if (!may_split || (M * O) % 4 != 0 || O % 4 != 0) return tp;
  const int wide = O > 128 ? 256 : (O > 64 ? 128 : 64);
  const int64_t tiles = ((M + kBM - 1) / kBM) * ((O + wide - 1) / wide);
  const int sms = num_sms();
  if (4 * tiles > sms) return tp;   // measured: a 2-3 way split costs more in the second pass than it gains
  int split = static_cast<int>(std::min<int64_t>(sms / tiles, kblocks / 4));
  if (split < 2) return tp;
  tp.bn = wide;
  tp.kper = static_cast<int>((kblocks + split - 1) / split);
  tp.ksplit = static_cast<int>((kblocks + tp.kper - 1) / tp.kper);
  tp.partial_bytes = round_up(static_cast<size_t>(tp.ksplit) * M * O * 4, 1024);
  return tp;
}

struct ConvPlan {
  bool tc = false;       // tensor-core path available
  bool prepass = false;  // needs channels-last copies in the workspace
  int64_t Cp = 0;
  size_t x_bytes = 0, w_bytes = 0;
  bool rowwin = false;   // few channels: row-window layout (always through the workspace)
  int64_t Hp = 0, Wpa = 0;
  // conv_rowrun: windows read in place from runs of the padded rows (pixels of 8 / Sw channels)
  // (C,H,W) items with 1x1 unpadded windows: the copy holds only the pixels the windows touch and is
  // then the [N*H'*W', Cp] matrix of a plain matrix product
  bool as_matrix = false;
  // (C,H,W) items with 1x1 unpadded windows whose rows the TMA unit can fetch (W a multiple of 8, at most 64): read
  // in place as a pixel-major (MN-major) A operand, no copy at all
  bool pixmajor = false;
  bool rowrun = false;
  int rr_cp = 0, rr_ksteps = 0, rr_bn = 0, rr_stages = 0, rr_raw_stages = 0, rr_nseg = 0;
  uint32_t rr_seg = 0, rr_slot = 0, rr_b_bytes = 0, rr_raw_seg = 0;
};

ConvPlan plan_conv(const DotProblem& d, uint32_t flags) {
  ConvPlan pl;
  pl.Cp = (d.C + 7) / 8 * 8;
  const bool fits = d.pw_lo <= 128 && d.ph_lo <= 128 && (d.Kw - 1 - d.pw_hi) <= 128 && (d.Kh - 1 - d.ph_hi) <= 128 &&
                    d.Kw <= 256 && d.Kh <= 256 && d.Sw <= 8 && d.Sh <= 8 && d.W < (1ll << 30) && d.H < (1ll << 30) &&
                    d.N < (1ll << 30) && d.M < (1ll << 31) && d.O < (1ll << 31) &&
                    d.Kh * d.Kw * pl.Cp < (1ll << 31);
  pl.tc = fits && ((d.M + 127) / 128) * ((d.O + 63) / 64) < (1ll << 28);
  pl.prepass = !d.channels_last || pl.Cp != d.C;
  // (with the fused squeeze + transpose the result rows are runs of W' pixels: whole 16-byte pieces)
  if (pl.tc && (!(flags & GL_OUT_NCHW) || (d.Wo * ((flags & GL_OUT_BF16) ? 2 : 4)) % 16 == 0) &&
      (d.Sw == 1 || d.Sw == 2 || d.Sw == 4 || d.Sw == 8) && d.C <= 8 / d.Sw &&
      d.O % ((flags & GL_OUT_BF16) ? 8 : 4) == 0 && d.O <= 128 && d.Kh <= 16 && d.Wo < (1ll << 24) &&
      d.N * d.Ho * ((d.Wo + kBM - 1) / kBM) < (1ll << 31) &&
      (d.N * d.C * d.H * d.W) % 8 == 0 &&                    // raw rows are copied as whole 16-byte pieces
      d.Kh * (d.channels_last ? 1 : d.C) <= 32) {            // one copy per lane of the copying warp
    const int cp = static_cast<int>(8 / d.Sw);
    const int ksteps = static_cast<int>((d.Kw * cp + 15) / 16);
    const int bn = static_cast<int>((d.O + 15) / 16 * 16);
    const uint32_t seg = 127 * 16 + ksteps * 32, slot = (seg + 127u) & ~127u;
    const uint32_t b_bytes = static_cast<uint32_t>(d.Kh) * ksteps * 2 * bn * 16;
    const int nseg = static_cast<int>(d.channels_last ? 1 : d.C);
    // a raw copy: the run's pixels as they lie in memory, widened to whole 16-byte pieces at both ends
    const uint32_t raw_seg = static_cast<uint32_t>(((seg / (2 * cp)) * (d.channels_last ? d.C : 1) * 2 + 30 + 15) / 16 * 16);
    const int64_t raw_stage = d.Kh * nseg * static_cast<int64_t>(raw_seg);
    const int64_t room = 113 * 1024 - 1024 - kRunEpiBytes - 256 - ((b_bytes + 127) & ~127u);   // two blocks per SM
    const int64_t stages = 3;                                                                   // tiles in flight
    const int64_t ring = d.Kh + (stages - 1) * d.Sh;                                            // widened runs kept
    const int64_t raw_stages = std::min<int64_t>(kRunMaxStages, (room - ring * slot) / raw_stage);
    if (raw_stages >= 2 && d.O * d.Kh * d.Kw * d.C * 2 <= ring * slot) {   // the weights fit the ring, where the block parks them once
      pl.rowrun = true;
      pl.prepass = false;   // the kernel reads both operands where they are, in either item layout
      pl.rr_cp = cp; pl.rr_ksteps = ksteps; pl.rr_bn = bn; pl.rr_stages = static_cast<int>(stages);
      pl.rr_seg = seg; pl.rr_slot = slot; pl.rr_b_bytes = b_bytes;
      pl.rr_raw_stages = static_cast<int>(raw_stages); pl.rr_nseg = nseg; pl.rr_raw_seg = raw_seg;
      return pl;
    }
  }
  if (pl.tc && pl.Cp < kBK && d.Kw * pl.Cp <= kBK && d.Wo < (1ll << 24) && d.N * (d.H + d.ph_lo + d.ph_hi) < (1ll << 31)) {
    pl.rowwin = true;
    pl.prepass = true;
    pl.Hp = d.H + d.ph_lo + d.ph_hi;
    // wide enough for the 64 values behind the last output column; a multiple of Sw (tensor-map stride rule)
    pl.Wpa = std::max(d.W + d.pw_lo + d.pw_hi, (d.Wo - 1) * d.Sw + kBK / pl.Cp);
    pl.Wpa = (pl.Wpa + d.Sw - 1) / d.Sw * d.Sw;
    pl.x_bytes = round_up(static_cast<size_t>(d.N * pl.Hp * pl.Wpa * pl.Cp) * 2, 1024);
    pl.w_bytes = round_up(static_cast<size_t>(d.O * d.Kh * kBK) * 2, 1024);
    return pl;
  }
  pl.pixmajor = pl.tc && !d.channels_last && d.Kh == 1 && d.Kw == 1 && d.ph_lo == 0 && d.ph_hi == 0 && d.pw_lo == 0 &&
                d.pw_hi == 0 && !(flags & GL_OUT_NCHW) && d.C % 8 == 0 && d.C >= kBK &&
                ((d.Sh == 1 && d.Sw == 1 && (d.H * d.W) % 8 == 0 && d.H * d.W < (1ll << 30)) ||   // one run of H*W pixels
                 (d.W % 8 == 0 && d.W <= 64 && (d.Sw == 1 || d.Sw == 2))) &&                     // row by row
                d.N * ((d.Ho + 1) / 2) < (1ll << 30);
  if (pl.pixmajor) {
    pl.prepass = false;
    return pl;
  }
  pl.as_matrix = pl.tc && !d.channels_last && d.Kh == 1 && d.Kw == 1 && d.ph_lo == 0 && d.ph_hi == 0 && d.pw_lo == 0 &&
                 d.pw_hi == 0 && !(flags & GL_OUT_NCHW) && pl.Cp >= kBK;
  if (pl.as_matrix) {
    pl.x_bytes = round_up(static_cast<size_t>(d.N * d.Ho * d.Wo * pl.Cp) * 2, 1024);
    pl.w_bytes = round_up(static_cast<size_t>(d.O * pl.Cp) * 2, 1024);
    return pl;
  }
  if (pl.prepass) {
    pl.x_bytes = round_up(static_cast<size_t>(d.N * d.H * d.W * pl.Cp) * 2, 1024);
    pl.w_bytes = round_up(static_cast<size_t>(d.O * d.Kh * d.Kw * pl.Cp) * 2, 1024);
  }
  return pl;
}

// Tiling of a stride-1 convolution for conv_halo.
struct HaloPlan {
  bool ok = false;
  int bn = 64, Wb = 0, R = 0, RB = 0, tiles_per_img = 0, sa = 0, sb = 0, resident = 0, tg = 1;
  int occ = 1;   // blocks per SM the shared-memory plan is made for
  int ctas = 1;  // 2: pairs of blocks share a column tile (each stages half of every weight box)
};

HaloPlan plan_halo(const DotProblem& d, const ConvPlan& pl, uint32_t flags) {
  HaloPlan hp;
  if (!d.conv || !pl.tc || pl.rowwin || (flags & GL_OUT_NCHW)) return hp;
  if (d.Sh != 1 || d.Sw != 1 || pl.Cp % kBK != 0 || d.O % ((flags & GL_OUT_BF16) ? 8 : 4) != 0) return hp;
  if (d.Kh == 1 && d.Kw == 1) return hp;   // no overlap between windows: nothing to keep
  const int64_t Wb = d.W + d.pw_lo + d.pw_hi;
  // the MMA of the last tap reads 128 rows starting (Kh-1)*Wb + Kw-1 rows into the stage
  if (Wb > 256 || (d.Kh - 1) * Wb + d.Kw - 1 + kBM > kHaloARows) return hp;
  const int64_t R = std::min<int64_t>(d.Ho, (kBM + d.Kw - 1) / Wb);
  if (R < 1) return hp;
  const int64_t tpi = (d.Ho + R - 1) / R;
  // rows of the 128-row tiles that hold real outputs; small images fill too little of a tile
  if (10 * d.Ho * d.Wo < 6 * tpi * kBM) return hp;
  if (d.N * tpi * ((d.O + 63) / 64) >= (1ll << 28) || d.N >= (1ll << 30) || d.H >= (1ll << 30)) return hp;
  hp.bn = d.O > 64 ? 128 : 64;
  hp.Wb = static_cast<int>(Wb);
  hp.R = static_cast<int>(R);
  hp.RB = static_cast<int>(R + d.Kh - 1);
  hp.tiles_per_img = static_cast<int>(tpi);
  // 128-wide tiles: pairs of blocks halve the weight bytes each SM pulls from L2 and the shared-memory
  // reads per MMA (measured 12.0 -> 11.2 us on 28x28x128, 11.7 -> 11.1 us on 14x14x256); at 64 columns the
  // pair's single block per SM loses to two independent blocks per SM
  if (hp.bn == 128 && d.N * tpi >= 2) hp.ctas = 2;
  // a B stage holds one filter row of one 64-channel chunk when that stays within 48 KB, else one tap
  hp.tg = d.Kw * hp.bn * kBK * 2 <= 48 * 1024 ? static_cast<int>(d.Kw) : 1;
  const int stage_b = hp.tg * (hp.bn / hp.ctas) * kBK * 2;
  const int64_t groups = (pl.Cp / kBK) * d.Kh * (d.Kw / hp.tg);
  const int tiles_n = static_cast<int>((d.O + hp.bn - 1) / hp.bn);
  if (hp.ctas == 2) {
    hp.occ = 1;
    hp.sa = 2;
    hp.sb = std::min<int>(kHaloMaxStages, (kHaloSmemBudget - hp.sa * kHaloAStage) / stage_b);
    hp.ok = hp.sb >= 2;
    return hp;
  }
  if (hp.bn == 64) {
    // two blocks per SM with one input-box stage each: start-up, loads and epilogue of one block run under
    // the MMAs of the other (one block per SM with resident weights measures the same, 14.7 against 14.4 us)
    hp.occ = 2;
    hp.sa = 1;
    hp.sb = std::min<int>(8, (113 * 1024 - 1024 - kHaloBarBytes - kHaloEpiBytes - kHaloAStage) / stage_b);
    hp.ok = hp.sb >= 2;
    return hp;
  }
  // weights that fit beside two input boxes stay in shared memory for the whole kernel
  if (tiles_n == 1 && groups <= kHaloMaxStages && groups * stage_b + 2 * kHaloAStage <= kHaloSmemBudget) {
    hp.resident = 1;
    hp.sb = static_cast<int>(groups);
    hp.sa = std::min<int>(6, (kHaloSmemBudget - hp.sb * stage_b) / kHaloAStage);
  } else {
    hp.sa = 2;
    hp.sb = std::min<int>(8, (kHaloSmemBudget - hp.sa * kHaloAStage) / stage_b);
    if (hp.sb > 4) { hp.sa = 3; hp.sb = std::min<int>(8, (kHaloSmemBudget - hp.sa * kHaloAStage) / stage_b); }
  }
  hp.ok = hp.sa >= 2 && hp.sb >= 2;
  return hp;
}

// Channels-last activations (N,H,W,Cp) as a tiled map whose box is the input block of one tile:
// 64 channels x Wb pixels x RB rows of one image; cells outside the image read as zeros.
bool encode_halo_box(CUtensorMap* m, const void* base, const DotProblem& d, int64_t Cp, int Wb, int RB) {
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(Cp), static_cast<cuuint64_t>(d.W), static_cast<cuuint64_t>(d.H),
                              static_cast<cuuint64_t>(d.N)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(Cp) * 2, static_cast<cuuint64_t>(d.W * Cp) * 2,
                                 static_cast<cuuint64_t>(d.H * d.W * Cp) * 2};
  const cuuint32_t box[4] = {kBK, static_cast<cuuint32_t>(Wb), static_cast<cuuint32_t>(RB), 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// (C,H,W) items as (W, H, C, N): one box = 64 pixels of one input row x 64 channels, landing channel by channel
// (128 bytes of pixels each): the MN-major A operand of 1x1 windows.  Pixels past W and channels past C read as zeros.
bool encode_chw_rows(CUtensorMap* m, const void* base, const DotProblem& d) {
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d.W), static_cast<cuuint64_t>(d.H), static_cast<cuuint64_t>(d.C),
                              static_cast<cuuint64_t>(d.N)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(d.W) * 2, static_cast<cuuint64_t>(d.H * d.W) * 2,
                                 static_cast<cuuint64_t>(d.C * d.H * d.W) * 2};
  const cuuint32_t box[4] = {64, 1, kBK, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// The same items as (H*W, C, N) when the windows touch every pixel: one box = 64 consecutive pixels x 64 channels.
bool encode_chw_flat(CUtensorMap* m, const void* base, const DotProblem& d) {
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(d.H * d.W), static_cast<cuuint64_t>(d.C), static_cast<cuuint64_t>(d.N)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(d.H * d.W) * 2, static_cast<cuuint64_t>(d.C * d.H * d.W) * 2};
  const cuuint32_t box[3] = {64, kBK, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Weights (O, Kh, Kw, Cp) viewed as (64 channels, O, chunk, tap): one box = BN rows x 64 channels of
// `tg` consecutive taps of one chunk, landing as [tap][row][64].
bool encode_halo_weights(CUtensorMap* m, const void* base, int64_t O, int64_t taps, int64_t Cp, int bn, int tg) {   // bn: rows per box
  const cuuint64_t dims[4] = {kBK, static_cast<cuuint64_t>(O), static_cast<cuuint64_t>(Cp / kBK),
                              static_cast<cuuint64_t>(taps)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(taps * Cp) * 2, kBK * 2, static_cast<cuuint64_t>(Cp) * 2};
  const cuuint32_t box[4] = {kBK, static_cast<cuuint32_t>(bn), 1, static_cast<cuuint32_t>(tg)};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return encode_tiled_cached(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

template <int BN, int OCC, int CTAS>
int launch_halo(const CUtensorMap& ma, const CUtensorMap& mb, float* out, const HaloParams& p, cudaStream_t st,
                const PreLaunch& pre) {
  const int smem = p.sa_stages * kHaloAStage + p.sb_stages * static_cast<int>(p.b_bytes) + kHaloEpiBytes + kHaloBarBytes + 1024;
  static bool attr_set_dev[64] = {false};
  static int max_pairs_dev[64] = {0};       // CTAS == 2: pairs that can be resident at once
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return GL_ERR_CUDA;
  if (!attr_set_dev[dev]) {
    if (cudaFuncSetAttribute(conv_halo<BN, OCC, CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             OCC == 2 ? 113 * 1024 : 232448) != cudaSuccess)
      return GL_ERR_CUDA;
    if (CTAS == 2) {
      // a persistent grid must not exceed what is resident at once (SMs pair up within a GPC)
      cudaLaunchConfig_t cfg;
      std::memset(&cfg, 0, sizeof(cfg));
      cudaLaunchAttribute cluster_attr;
      std::memset(&cluster_attr, 0, sizeof(cluster_attr));
      cluster_attr.id = cudaLaunchAttributeClusterDimension;
      cluster_attr.val.clusterDim.x = 2;
      cluster_attr.val.clusterDim.y = 1;
      cluster_attr.val.clusterDim.z = 1;
      cfg.gridDim = dim3(static_cast<unsigned>(OCC * (num_sms() / 2 * 2)));
      cfg.blockDim = dim3(kTcThreads);
      cfg.dynamicSmemBytes = OCC == 2 ? 113 * 1024 : 232448;
      cfg.attrs = &cluster_attr;
      cfg.numAttrs = 1;
      int pairs = 0;
      if (cudaOccupancyMaxActiveClusters(&pairs, conv_halo<BN, OCC, CTAS>, &cfg) != cudaSuccess || pairs < 1)
        return GL_ERR_CUDA;
      max_pairs_dev[dev] = pairs;
    }
    attr_set_dev[dev] = true;
  }
  const int tiles = p.tiles_m * p.tiles_n;
  if (const int rc = run_pre(pre)) return rc;
  if (CTAS == 2) {
    const int pairs = std::min(tiles, std::min(max_pairs_dev[dev], OCC * (num_sms() / 2)));
    return launch_pdl(conv_halo<BN, OCC, CTAS>, dim3(static_cast<unsigned>(2 * pairs)), dim3(kTcThreads),
                      static_cast<size_t>(smem), st, 2, ma, mb, out, p) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  }
  const int grid = std::min(tiles, OCC * num_sms());
  return launch_pdl(conv_halo<BN, OCC, CTAS>, dim3(static_cast<unsigned>(grid)), dim3(kTcThreads), static_cast<size_t>(smem), st, 1,
                    ma, mb, out, p) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
}

int run_halo(const HaloPlan& hp, const DotProblem& d, int64_t Cp, const uint16_t* x, const uint16_t* wt, float* out,
             int relu, int out_bf16, cudaStream_t st, const PreLaunch& pre) {
  HaloParams p;
  std::memset(&p, 0, sizeof(p));
  p.O = d.O; p.relu = relu; p.out_bf16 = out_bf16;
  p.N = static_cast<int>(d.N);
  p.Ho = static_cast<int>(d.Ho); p.Wo = static_cast<int>(d.Wo);
  p.Wb = hp.Wb; p.R = hp.R;
  p.tiles_m = (static_cast<int>(d.N) * hp.tiles_per_img + hp.ctas - 1) / hp.ctas;
  p.tiles_n = static_cast<int>((d.O + hp.bn - 1) / hp.bn);
  p.Kh = static_cast<int>(d.Kh); p.Kw = static_cast<int>(d.Kw);
  p.Cp = static_cast<int>(Cp);
  p.cchunks = static_cast<int>(Cp / kBK);
  p.tg = hp.tg;
  p.groups_per_chunk = p.Kh * (p.Kw / hp.tg);
  p.ph = static_cast<int>(d.ph_lo); p.pw = static_cast<int>(d.pw_lo);
  p.sa_stages = hp.sa; p.sb_stages = hp.sb; p.b_resident = hp.resident;
  p.prefetch = pre ? 0 : 1;
  p.a_bytes = static_cast<uint32_t>(kBK * 2 * hp.Wb * hp.RB);
  p.b_bytes = static_cast<uint32_t>(hp.tg * (hp.bn / hp.ctas) * kBK * 2);
  p.div_tiles_n.set(p.tiles_n);
  p.div_tpi.set(hp.tiles_per_img);
  p.div_wb.set(hp.Wb);
  CUtensorMap ma, mb;
  if (!encode_halo_box(&ma, x, d, Cp, hp.Wb, hp.RB) ||
      !encode_halo_weights(&mb, wt, d.O, d.Kh * d.Kw, Cp, hp.bn / hp.ctas, hp.tg))
    return GL_ERR_CUDA;
  if (hp.ctas == 2) return launch_halo<128, 1, 2>(ma, mb, out, p, st, pre);
  return hp.bn == 128 ? launch_halo<128, 1, 1>(ma, mb, out, p, st, pre) : launch_halo<64, 2, 1>(ma, mb, out, p, st, pre);
}

// A 1x1, stride-1, unpadded window over channels-last items is no window at all: the activations
// already are the [N*H*W, C] matrix (the special case "1x1 conv == matmul").
bool conv_is_plain_matrix(const DotProblem& d, uint32_t flags) {
  return d.conv && d.channels_last && d.Kh == 1 && d.Kw == 1 && d.Sh == 1 && d.Sw == 1 && d.ph_lo == 0 &&
         d.ph_hi == 0 && d.pw_lo == 0 && d.pw_hi == 0 && d.C % 8 == 0 && !(flags & GL_OUT_NCHW);
}

// The kernel counts tiles in 32-bit integers.
bool tile_count_ok(const DotProblem& d) { return ((d.M + 127) / 128) * ((d.O + 63) / 64) < (1ll << 28); }

bool dense_tc_ok(const DotProblem& d) {
  return !d.conv && !d.general && d.K % 8 == 0 && d.M < (1ll << 31) && d.O < (1ll << 31) && d.K < (1ll << 31) &&
         tile_count_ok(d);
}

void fill_general(const gl_ap* a0, const gl_windows* w, const DotProblem& d, GenA* g) {
  std::memset(g, 0, sizeof(*g));
  g->M = d.M; g->K = d.K; g->O = d.O;
  g->HoWo = d.conv ? d.Ho * d.Wo : 1;
  if (!w) { g->mode = 0; return; }
  if (d.conv) {
    g->mode = 1;
    g->channels_last = d.channels_last;
    g->C = d.C; g->H = d.H; g->W = d.W; g->Kh = d.Kh; g->Kw = d.Kw; g->Sh = d.Sh; g->Sw = d.Sw;
    g->ph = d.ph_lo; g->pw = d.pw_lo; g->Ho = d.Ho; g->Wo = d.Wo;
    return;
  }
  g->mode = 2;
  g->n = w->n;
  const int na = a0->access_ndim;
  int64_t s = 1;
  for (int i = w->n - 1; i >= 0; --i) {
    const int64_t b = a0->shape[na + i];
    g->in_size[i] = b;
    g->in_stride[i] = s;
    s *= b;
    g->w[i] = w->wshape[i];
    g->s[i] = w->stride[i];
    g->pad_lo[i] = w->pad_lo[i];
    g->out_ext[i] = (b + w->pad_lo[i] + w->pad_hi[i] - (w->wshape[i] - 1) + w->stride[i] - 1) / w->stride[i];
  }
  g->item = s;
}


// Scratch of a call in two parts: the layout copies, without which it cannot run, and the partial planes of a
// split contraction, without which it runs unsplit.
void workspace_parts(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, uint32_t flags, size_t* required,
                     size_t* optional) {
  *required = *optional = 0;
  DotProblem d;
  if (classify_dot(a0, w, a1, &d) != GL_OK) return;
  if (flags & GL_DOT_GENERAL_KERNEL) return;
  if (conv_is_plain_matrix(d, flags)) d.conv = false;
  if (!d.conv) {
    if (dense_tc_ok(d)) *optional = plan_tiles(d.M, d.O, (d.K + kBK - 1) / kBK, true).partial_bytes;
    return;
  }
  const ConvPlan pl = plan_conv(d, flags);
  if (!pl.tc) return;
  *required = pl.prepass ? pl.x_bytes + pl.w_bytes : 0;
  // the resident-window and row-run kernels never split
  if (!pl.rowwin && !pl.rowrun && pl.Cp >= kBK && !(flags & GL_OUT_NCHW) && !plan_halo(d, pl, flags).ok)
    *optional = plan_tiles(d.M, d.O, d.Kh * d.Kw * ((pl.Cp + kBK - 1) / kBK), true).partial_bytes;
}

}  // namespace

extern "C" {

size_t gl_cartesian_dot_workspace(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, uint32_t flags) {
  size_t required = 0, optional = 0;
  workspace_parts(a0, w, a1, flags, &required, &optional);
  return required + optional;
}

int gl_cartesian_dot(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, gl_ap* out, uint32_t flags,
                     void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_data(a0);
  if (rc) return rc;
  rc = check_data(a1);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (a0->dtype != GL_BF16 || a1->dtype != GL_BF16) return GL_ERR_DTYPE;
  if (flags & ~(GL_EPILOGUE_RELU | GL_DOT_GENERAL_KERNEL | GL_OUT_NCHW | GL_OUT_BF16)) return GL_ERR_UNSUPPORTED;
  const int out_nchw = (flags & GL_OUT_NCHW) ? 1 : 0;
  const int out_bf16 = (flags & GL_OUT_BF16) ? 1 : 0;
  DotProblem d;
  rc = classify_dot(a0, w, a1, &d);
  if (rc) return rc;
  gl_ap want = *out;
  rc = out_nchw ? gl_shape_cartesian_dot_nchw(a0, w, a1, &want) : gl_shape_cartesian_dot(a0, w, a1, &want);
  if (rc) return rc;
  if (out_bf16) want.dtype = GL_BF16;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int relu = (flags & GL_EPILOGUE_RELU) ? 1 : 0;
  float* dst = static_cast<float*>(out->data);
  const uint16_t* pa = static_cast<const uint16_t*>(a0->data);
  const uint16_t* pb = static_cast<const uint16_t*>(a1->data);

  const bool force_general = (flags & GL_DOT_GENERAL_KERNEL) != 0;
  if (!force_general && conv_is_plain_matrix(d, flags)) d.conv = false;
  ConvPlan pl;
  if (d.conv) pl = plan_conv(d, flags);
  const bool use_tc = !force_general && ((d.conv && pl.tc) || dense_tc_ok(d));
  if (!use_tc) {
    GenA g;
    fill_general(a0, w, d, &g);
    g.out_nchw = out_nchw;
    g.out_bf16 = out_bf16;
    const int64_t gx = (d.M + 63) / 64, gy = (d.O + 63) / 64;
    if (gy > 65535 || gx > 0x7FFFFFFF) return GL_ERR_UNSUPPORTED;
    dot_general<<<dim3(static_cast<unsigned>(gx), static_cast<unsigned>(gy)), 256, 0, st>>>(pa, pb, dst, g, relu);
    return cudaGetLastError() == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  }
  if (!driver_api().ok) return GL_ERR_CUDA;

  TcParams p;
  std::memset(&p, 0, sizeof(p));
  p.M = d.M; p.O = d.O; p.relu = relu;
  p.out_nchw = out_nchw;
  // tile width and K split; a K split needs room for its partial planes behind the layout copies
  const size_t pre_bytes = (d.conv && pl.prepass) ? pl.x_bytes + pl.w_bytes : 0;
  HaloPlan hp;
  if (d.conv) hp = plan_halo(d, pl, flags);
  const bool split_mode = (!d.conv || (!pl.rowwin && pl.Cp >= kBK)) && !out_nchw && !hp.ok && !pl.pixmajor;
  const int64_t kblocks_all = !d.conv ? (d.K + kBK - 1) / kBK : d.Kh * d.Kw * ((pl.Cp + kBK - 1) / kBK);
  TilePlan tp = plan_tiles(d.M, d.O, kblocks_all, split_mode);
  if (tp.ksplit > 1 && (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 1023u) ||
                        workspace_bytes < pre_bytes + tp.partial_bytes))
    tp = plan_tiles(d.M, d.O, kblocks_all, false);
  const int bn = tp.bn;
  p.ksplit = tp.ksplit;
  p.kper = tp.kper;
  float* const final_dst = dst;
  p.out_bf16 = out_bf16;
  if (tp.ksplit > 1) {   // fp32 partial planes; relu and the rounding to bf16 happen in the summing kernel
    dst = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + pre_bytes);
    p.relu = 0;
    p.out_bf16 = 0;
  }
  // the launch of the partial-sum kernel when the contraction was split
  auto finish = [&](int rc_launch) -> int {
    if (rc_launch != GL_OK || tp.ksplit == 1) return rc_launch;
    const int64_t n = d.M * d.O;
    return launch_pdl(splitk_reduce, dim3(static_cast<unsigned>(std::min<int64_t>((n / 4 + 255) / 256, 148 * 8))), dim3(256),
                      0, st, 1, static_cast<const float*>(dst), final_dst, n, tp.ksplit, relu, out_bf16) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  };
  p.tiles_m = static_cast<int>((d.M + kBM - 1) / kBM);
  p.tiles_n = static_cast<int>((d.O + bn - 1) / bn);
  CUtensorMap ma, mb;

  if (!d.conv) {
    p.K = d.K;
    p.kblocks = static_cast<int>((d.K + kBK - 1) / kBK);
    if (!encode_kmajor_sw128(&ma, pa, d.M, d.K, kBM) ||
        !encode_kmajor_sw128(&mb, pb, d.O, d.K, use_pair(kDense, bn, p) ? bn / 4 : bn))
      return GL_ERR_CUDA;
    return finish(launch_tc_bn<kDense>(bn, ma, mb, dst, p, st, PreLaunch()));
  }

  const uint16_t* x = pa;
  const uint16_t* wt = pb;
  PreLaunch pre;   // the layout copies, enqueued by the launch function once nothing else can fail
  if (pl.rowrun) {
    RowRunParams rp;
    std::memset(&rp, 0, sizeof(rp));
    rp.O = d.O; rp.relu = relu; rp.out_bf16 = out_bf16; rp.out_nchw = out_nchw;
    rp.C = static_cast<int>(d.C); rp.H = static_cast<int>(d.H); rp.W = static_cast<int>(d.W);
    rp.Ho = static_cast<int>(d.Ho); rp.Wo = static_cast<int>(d.Wo);
    rp.Sh = static_cast<int>(d.Sh); rp.Sw = static_cast<int>(d.Sw);
    rp.Kh = static_cast<int>(d.Kh); rp.Kw = static_cast<int>(d.Kw);
    rp.ph = static_cast<int>(d.ph_lo); rp.pw = static_cast<int>(d.pw_lo);
    while ((1 << rp.cp_log2) < pl.rr_cp) ++rp.cp_log2;
    rp.channels_last = d.channels_last ? 1 : 0;
    rp.xs_n = d.C * d.H * d.W;
    if (d.channels_last) { rp.xs_h = d.W * d.C; rp.xs_c = 1; }
    else { rp.xs_h = d.W; rp.xs_c = d.H * d.W; }
    rp.div_bn.set(pl.rr_bn);
    rp.nseg = pl.rr_nseg;
    rp.raw_seg_bytes = pl.rr_raw_seg;
    rp.raw_row_bytes = pl.rr_raw_seg * static_cast<uint32_t>(pl.rr_nseg);
    rp.raw_stage_bytes = rp.raw_row_bytes * static_cast<uint32_t>(d.Kh);
    rp.raw_stages = pl.rr_raw_stages;
    rp.w_elems = static_cast<int>(d.O * d.Kh * d.Kw * d.C);
    rp.div_nseg.set(pl.rr_nseg);
    rp.segs = static_cast<int>((d.Wo + kBM - 1) / kBM);
    rp.tiles = static_cast<int>(d.N * d.Ho * rp.segs);
    rp.ksteps = pl.rr_ksteps; rp.bn = pl.rr_bn;
    rp.seg_bytes = pl.rr_seg; rp.slot_bytes = pl.rr_slot;
    rp.b_bytes = pl.rr_b_bytes;
    rp.stages = pl.rr_stages;
    rp.ring = static_cast<int>(d.Kh + (pl.rr_stages - 1) * d.Sh);
    // strips: about one per block slot (two blocks per SM)
    rp.strip = static_cast<int>(std::max<int64_t>(1, (static_cast<int64_t>(rp.tiles) + 2 * num_sms() - 1) / (2 * num_sms())));
    rp.strips_per_img = static_cast<int>((d.Ho + rp.strip - 1) / rp.strip);
    rp.div_spi.set(rp.strips_per_img);
    rp.div_ring.set(rp.ring);
    rp.div_segs.set(rp.segs);
    rp.div_ho.set(d.Ho);
    CUtensorMap mc;
    if (out_nchw ? !encode_result_nchw(&mc, dst, d.N, d.O, d.Ho, d.Wo, out_bf16 != 0)
                 : !encode_result_rows(&mc, dst, d.N * d.Ho, d.Wo, d.O, out_bf16 != 0))
      return GL_ERR_CUDA;
    const int smem = 1024 + kRunEpiBytes + static_cast<int>((rp.b_bytes + 127u) & ~127u) +
                     rp.ring * static_cast<int>(rp.slot_bytes) + rp.raw_stages * static_cast<int>(rp.raw_stage_bytes) + 256;
    static bool attr_set_dev[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return GL_ERR_CUDA;
    if (!attr_set_dev[dev]) {
      if (cudaFuncSetAttribute(conv_rowrun<0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024) != cudaSuccess ||
          cudaFuncSetAttribute(conv_rowrun<3, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024) != cudaSuccess ||
          cudaFuncSetAttribute(conv_rowrun<3, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024) != cudaSuccess)
        return GL_ERR_CUDA;
      attr_set_dev[dev] = true;
    }
    const int64_t grid = d.N * rp.segs * rp.strips_per_img;   // one strip per block
    if (grid >= (1ll << 31)) return GL_ERR_UNSUPPORTED;
    // three channels (RGB) have kernels of their own, one per item layout
    auto kernel = d.C == 3 ? (d.channels_last ? conv_rowrun<3, 1> : conv_rowrun<3, 0>) : conv_rowrun<0, 0>;
    return launch_pdl(kernel, dim3(static_cast<unsigned>(grid)), dim3(kRunThreads), static_cast<size_t>(smem), st, 1,
                      pa, pb, mc, rp) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  }
  if (pl.pixmajor) {
    // 1x1 windows of (C,H,W) items: A tiles come straight from the items, pixel-major; the weights (O, C, 1, 1)
    // already are the [O, C] matrix.  With Sw = 2 the odd pixels of a row are multiplied too and dropped.
    p.K = d.C;
    p.kblocks = static_cast<int>((d.C + kBK - 1) / kBK);
    p.Sh = static_cast<int>(d.Sh); p.Sw = static_cast<int>(d.Sw);
    p.Ho = static_cast<int>(d.Ho); p.Wo = static_cast<int>(d.Wo);
    p.pix_w = static_cast<int>(d.W);
    p.pix_flat = (d.Sh == 1 && d.Sw == 1 && (d.H * d.W) % 8 == 0) ? 1 : 0;
    p.pix_hw = static_cast<int>(d.H * d.W);
    p.pix_tpi = static_cast<int>(p.pix_flat ? (d.H * d.W + kBM - 1) / kBM : (d.Ho + 1) / 2);
    p.tiles_m = static_cast<int>(d.N * p.pix_tpi);
    p.tiles_n = static_cast<int>((d.O + 127) / 128);
    if (!(p.pix_flat ? encode_chw_flat(&ma, pa, d) : encode_chw_rows(&ma, pa, d)) || !encode_kmajor_sw128(&mb, pb, d.O, d.C, 128))
      return GL_ERR_CUDA;
    return launch_tc<128, kChwPix, 1, 1>(ma, mb, dst, p, st, PreLaunch());
  }
  if (pl.prepass) {
    const size_t need = pl.x_bytes + pl.w_bytes;
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 1023u)) return GL_ERR_WORKSPACE;
    uint16_t* xs = static_cast<uint16_t*>(workspace);
    uint16_t* ws = reinterpret_cast<uint16_t*>(static_cast<unsigned char*>(workspace) + pl.x_bytes);
    if (pl.rowwin) {
      pre = [=]() -> int {
        rowwin_pack_x<<<static_cast<unsigned>(d.N * pl.Hp), 256, 0, st>>>(
            pa, xs, d.channels_last ? 1 : 0, static_cast<int>(d.C), static_cast<int>(d.H), static_cast<int>(d.W),
            static_cast<int>(pl.Hp), static_cast<int>(pl.Wpa), static_cast<int>(pl.Cp), static_cast<int>(d.ph_lo),
            static_cast<int>(d.pw_lo));
        rowwin_pack_w<<<static_cast<unsigned>(std::min<int64_t>((d.O * d.Kh * 64 + 255) / 256, 1 << 20)), 256, 0, st>>>(
            pb, ws, d.channels_last ? 1 : 0, d.O, d.C, d.Kh, d.Kw, static_cast<int>(pl.Cp));
        return cudaGetLastError() == cudaSuccess ? GL_OK : GL_ERR_CUDA;
      };
      p.K = d.Kh * kBK;
      p.kblocks = static_cast<int>(d.Kh);
      p.Cp = static_cast<int>(pl.Cp);
      p.Kh = static_cast<int>(d.Kh); p.Kw = static_cast<int>(d.Kw);
      p.Sh = static_cast<int>(d.Sh); p.Sw = static_cast<int>(d.Sw);
      p.Ho = static_cast<int>(d.Ho); p.Wo = static_cast<int>(d.Wo);
      p.Hp = static_cast<int>(pl.Hp);
      p.segs = static_cast<int>((d.Wo + kBM - 1) / kBM);
      p.tiles_m = static_cast<int>(d.N * d.Ho * p.segs);
      if (encode_rowwin(&ma, xs, d.N * pl.Hp, d.Wo, pl.Wpa, pl.Cp, d.Sw) &&
          encode_kmajor_sw128(&mb, ws, d.O, p.K, bn))
        return launch_tc_bn<kRowWin>(bn, ma, mb, dst, p, st, pre);
      return GL_ERR_CUDA;
    }
    const int64_t HW = d.H * d.W, T = d.Kh * d.Kw;
    if (d.channels_last) {
      // (N,H,W,C) with C not a multiple of 8: re-pitch the channel dim (a (N*HW, C) -> (N*HW, Cp) copy)
      pre = [=]() -> int {
        weights_to_channels_last<<<static_cast<unsigned>(std::min<int64_t>((d.N * HW * pl.Cp + 255) / 256, 1 << 20)), 256, 0,
                                   st>>>(pa, xs, d.N * HW, d.C, 1, pl.Cp);
        weights_to_channels_last<<<static_cast<unsigned>(std::min<int64_t>((d.O * T * pl.Cp + 255) / 256, 1 << 20)), 256, 0,
                                   st>>>(pb, ws, d.O * T, d.C, 1, pl.Cp);
        return cudaGetLastError() == cudaSuccess ? GL_OK : GL_ERR_CUDA;
      };
    } else {
      PrepassParams pp;
      std::memset(&pp, 0, sizeof(pp));
      pp.C = static_cast<int>(d.C); pp.H = static_cast<int>(d.H); pp.W = static_cast<int>(d.W);
      pp.Cp = static_cast<int>(pl.Cp);
      pp.Hs = static_cast<int>(pl.as_matrix ? d.Ho : d.H); pp.Ws = static_cast<int>(pl.as_matrix ? d.Wo : d.W);
      pp.Sh = static_cast<int>(pl.as_matrix ? d.Sh : 1); pp.Sw = static_cast<int>(pl.as_matrix ? d.Sw : 1);
      pp.O = static_cast<int>(d.O); pp.T = static_cast<int>(T);
      pp.total_pix = d.N * pp.Hs * pp.Ws;
      const int64_t tiles_p = (pp.total_pix + 63) / 64, tiles_c = (pl.Cp + 63) / 64;
      // weights of 1x1 windows with an unpadded channel count already are the [O, C] matrix: no copy
      const bool copy_w = !(T == 1 && pl.Cp == d.C);
      const int wwarps = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(8, (32 * 1024) / (64 * T * 2))));
      const int64_t x_blocks = tiles_p * tiles_c, w_blocks = copy_w ? (d.O * tiles_c + wwarps - 1) / wwarps : 0;
      if (T <= 256 && x_blocks + w_blocks < (1ll << 31) && d.H * d.W < (1ll << 31) && d.C < (1ll << 24)) {
        pp.tiles_c = static_cast<int>(tiles_c);
        pp.wtiles_c = static_cast<int>(tiles_c);
        pp.wwarps = wwarps;
        pp.x_blocks = static_cast<int>(x_blocks);
        pp.fast = pp.total_pix + 64 < (1ll << 31) ? 1 : 0;
        pp.by_tiles_c = make_fastdiv(tiles_c);
        pp.by_npix = make_fastdiv(static_cast<int64_t>(pp.Hs) * pp.Ws);
        pp.by_Ws = make_fastdiv(pp.Ws);
        if (!copy_w) ws = const_cast<uint16_t*>(pb);
        const size_t smem = std::max<size_t>(64 * 66 * 2, static_cast<size_t>(wwarps) * 64 * T * 2);
        uint16_t* const ws_dst = ws;
        pre = [=]() -> int {
          return launch_pdl(nchw_prepass, dim3(static_cast<unsigned>(x_blocks + w_blocks)), dim3(256), smem, st, 1, pa, xs, pb,
                            ws_dst, pp) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
        };
      } else if (pl.as_matrix) {
        return GL_ERR_UNSUPPORTED;
      } else {
        if (d.N > 65535 || (d.C + 31) / 32 > 65535) return GL_ERR_UNSUPPORTED;
        const dim3 grid(static_cast<unsigned>((HW + 31) / 32), static_cast<unsigned>((pl.Cp + 31) / 32),
                        static_cast<unsigned>(d.N));
        pre = [=]() -> int {
          nchw_to_nhwc_pad<<<grid, 256, 0, st>>>(pa, xs, d.C, HW, pl.Cp);
          weights_to_channels_last<<<static_cast<unsigned>(std::min<int64_t>((d.O * T * pl.Cp + 255) / 256, 1 << 20)), 256,
                                     0, st>>>(pb, ws, d.O, d.C, T, pl.Cp);
          return cudaGetLastError() == cudaSuccess ? GL_OK : GL_ERR_CUDA;
        };
      }
    }
    x = xs;
    wt = ws;
  }
  const int64_t Cp = pl.Cp, taps = d.Kh * d.Kw;
  if (pl.as_matrix) {   // the copy is the [M, Cp] matrix, the weights [O, Cp]
    p.K = Cp;
    p.kblocks = static_cast<int>((Cp + kBK - 1) / kBK);
    if (!encode_kmajor_sw128(&ma, x, d.M, Cp, kBM) ||
        !encode_kmajor_sw128(&mb, wt, d.O, Cp, use_pair(kDense, bn, p) ? bn / 4 : bn))
      return GL_ERR_CUDA;
    return finish(launch_tc_bn<kDense>(bn, ma, mb, dst, p, st, pre));
  }
  if (hp.ok) return run_halo(hp, d, Cp, x, wt, dst, relu, out_bf16, st, pre);
  p.K = taps * Cp;
  p.Cp = static_cast<int>(Cp);
  p.Kh = static_cast<int>(d.Kh); p.Kw = static_cast<int>(d.Kw);
  p.Sh = static_cast<int>(d.Sh); p.Sw = static_cast<int>(d.Sw);
  p.ph = static_cast<int>(d.ph_lo); p.pw = static_cast<int>(d.pw_lo);
  p.Ho = static_cast<int>(d.Ho); p.Wo = static_cast<int>(d.Wo);
  if (Cp >= kBK) {
    p.cchunks = static_cast<int>((Cp + kBK - 1) / kBK);
    p.kblocks = static_cast<int>(taps) * p.cchunks;
    if (!encode_im2col(&ma, x, d, Cp, kBK, true) ||
        !encode_kmajor_sw128(&mb, wt, d.O, p.K, use_pair(kIm2col, bn, p) ? bn / 4 : bn))
      return GL_ERR_CUDA;
    return finish(launch_tc_bn<kIm2col>(bn, ma, mb, dst, p, st, pre));
  }
  p.cchunks = static_cast<int>(Cp / 8);
  p.kblocks = static_cast<int>((taps * p.cchunks + 7) / 8);
  if (!encode_im2col(&ma, x, d, Cp, 8, false) || !encode_kmajor_granules(&mb, wt, d.O, p.K, bn)) return GL_ERR_CUDA;
  return launch_tc_bn<kIm2colGranule>(bn, ma, mb, dst, p, st, pre);
}

int gl_selftest_bounded_wait(uint32_t limit_ms, void* stream) {
  if (limit_ms < 1 || limit_ms > 1000) return GL_ERR_SHAPE;
  bounded_wait_selftest<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<uint64_t>(limit_ms) * 1000000ull);
  return cudaGetLastError() == cudaSuccess ? GL_OK : GL_ERR_CUDA;
}

int gl_poll_device_status(void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned int v = 0;
  if (cudaStreamSynchronize(st) != cudaSuccess) return GL_ERR_CUDA;
  if (cudaMemcpyFromSymbol(&v, g_status, sizeof(v)) != cudaSuccess) return GL_ERR_CUDA;
  if (v) {
    const unsigned int zero = 0;
    if (cudaMemcpyToSymbol(g_status, &zero, sizeof(zero)) != cudaSuccess) return GL_ERR_CUDA;
    return GL_ERR_TIMEOUT;
  }
  return GL_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------
// gl_cartesian_dot_static: the same operation for callers that cannot allocate
// ------------------------------------------------------------------------
//
// gl_cartesian_dot needs a caller-supplied workspace when the activations come
// in the (C,H,W) item layout (or with a channel count that is not a multiple
// of 8): the channels-last copies live there.  Some hosts of this library have
// no way to obtain that memory - code running inside a framework's operator
// where the allocator is off limits, a plug-in that is only handed its input
// and output buffers, a process that has given all device memory to a pool.
// For them the scratch is a fixed array inside the library image.  Every GPU
// that loads the library holds these bytes until the process exits.

// GL_STATIC_SCRATCH_BYTES (gl.h) is what a call may use; 1024 more bytes absorb the alignment.
static __device__ __align__(256) unsigned char g_static_scratch[GL_STATIC_SCRATCH_BYTES + 1024];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// In host code `g_static_scratch` is only a handle for the runtime, not a
// device address, so the address is asked for once per device (with that
// device current) and remembered.
int static_scratch_address(void** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GL_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return GL_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *ptr = g_scratch_addr[dev];
  return GL_OK;
}

}  // namespace

extern "C" {

int gl_cartesian_dot_static(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, gl_ap* out, uint32_t flags,
                            void* stream) {
  // validate first, so that an over-sized request is told apart from a malformed one
  int rc = check_data(a0);
  if (rc) return rc;
  rc = check_data(a1);
  if (rc) return rc;
  if (a0->dtype != GL_BF16 || a1->dtype != GL_BF16) return GL_ERR_DTYPE;
  DotProblem d;
  rc = classify_dot(a0, w, a1, &d);
  if (rc) return rc;
  // only the layout copies must fit: a contraction whose partial planes do not fit beside them runs unsplit
  size_t required = 0, optional = 0;
  workspace_parts(a0, w, a1, flags, &required, &optional);
  if (required > GL_STATIC_SCRATCH_BYTES) return GL_ERR_WORKSPACE;   // beyond the built-in scratch
  void* base = nullptr;
  rc = static_scratch_address(&base);
  if (rc) return rc;
  // the array is 256-byte aligned; the tensor maps want 1024
  const uintptr_t aligned = (reinterpret_cast<uintptr_t>(base) + 1023u) & ~static_cast<uintptr_t>(1023u);
  return gl_cartesian_dot(a0, w, a1, out, flags, reinterpret_cast<void*>(aligned), GL_STATIC_SCRATCH_BYTES, stream);
}

}  // extern "C"
