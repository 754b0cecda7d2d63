// Memory-bound access-pattern kernels: materialised `windows` (im2col),
// `transpose`, `pad` (transformer table, Section 4.2; pad is the constant
// border added for ML workloads), and the operators `reduceMax` and `relu`
// under `compute` (Section 4.3).  These move or compare values, so every
// result is bit-exact.  Each kernel is bounded by HBM bandwidth: coalesced
// 128-bit global accesses, shared-memory staging where the access pattern
// would otherwise scatter.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>

#include "gl_internal.h"
#include "gl_launch.cuh"

using namespace gl;

namespace {

constexpr int kThreads = 256;

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? GL_OK : GL_ERR_CUDA; }

inline unsigned grid_for(int64_t work_items, int per_block) {
  int64_t g = (work_items + per_block - 1) / per_block;
  return static_cast<unsigned>(g < 1 ? 1 : g);
}

template <typename T> struct Fill;
template <> struct Fill<uint32_t> {
  static __host__ __device__ uint32_t value(int kind) { return kind == GL_PAD_NEG_INF ? 0xFF800000u : 0u; }
};
template <> struct Fill<uint16_t> {
  static __host__ __device__ uint16_t value(int kind) { return kind == GL_PAD_NEG_INF ? 0xFF80u : 0u; }
};

// ------------------------------------------------------------------------
// transpose
// ------------------------------------------------------------------------

struct BatchDims {
  int n;
  int64_t size[GL_MAX_DIMS];
  int64_t in_stride[GL_MAX_DIMS];
  int64_t out_stride[GL_MAX_DIMS];
};

struct TileParams {
  int64_t sizeA, sizeB;        // A: contiguous in the input, B: contiguous in the output
  int64_t in_strideB, out_strideA;
  int64_t tilesA, tilesB;
  BatchDims batch;
};

// idx is a block index (below 2^32, and so is every extent whose product bounds it): 32-bit divisions,
// a fifth of the instructions of 64-bit ones, which matters for blocks that move one 16 KB tile.
__device__ __forceinline__ void batch_offsets(const BatchDims& b, uint32_t idx, int64_t& in_off, int64_t& out_off) {
  in_off = 0;
  out_off = 0;
#pragma unroll 1
  for (int d = b.n - 1; d >= 0; --d) {
    const uint32_t size = static_cast<uint32_t>(b.size[d]);
    const uint32_t q = idx / size;
    const int64_t i = idx - q * size;
    idx = q;
    in_off += i * b.in_stride[d];
    out_off += i * b.out_stride[d];
  }
}

// 2D tile transpose with 128-bit accesses on both sides.  Each thread loads a
// VEC x VEC block (VEC rows of one 16-byte vector), transposes it in registers
// and parks it in shared memory with an XOR swizzle on the vector index, so
// that both the writes and the later row reads are free of bank conflicts.
template <typename T, int VEC>
__global__ void __launch_bounds__(kThreads) transpose_tiled_vec(const T* __restrict__ in, T* __restrict__ out,
                                                                const TileParams p) {
  constexpr int TILE = 16 * VEC;
  __shared__ uint4 tile[TILE][16];
  pdl_wait();
  pdl_launch_dependents();
  uint32_t bid = blockIdx.x;   // tilesA * tilesB * batch = the grid size: every factor is below 2^32
  const uint32_t nA = static_cast<uint32_t>(p.tilesA), nB = static_cast<uint32_t>(p.tilesB);
  const uint32_t qA = bid / nA;
  const int64_t tileA = bid - qA * nA;
  bid = qA;
  const uint32_t qB = bid / nB;
  const int64_t tileB = bid - qB * nB;
  bid = qB;
  int64_t in_off, out_off;
  batch_offsets(p.batch, bid, in_off, out_off);
  const int ta = threadIdx.x & 15, tb = threadIdx.x >> 4;
  const int64_t a0 = tileA * TILE, b0 = tileB * TILE;

  union Row { uint4 v; T e[VEC]; };
  Row blk[VEC];
  {
    const int64_t a = a0 + ta * VEC;
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
      const int64_t b = b0 + tb * VEC + i;
      if (a < p.sizeA && b < p.sizeB)
        blk[i].v = *reinterpret_cast<const uint4*>(in + in_off + b * p.in_strideB + a);
      else
        blk[i].v = make_uint4(0, 0, 0, 0);
    }
  }
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    Row r;
#pragma unroll
    for (int i = 0; i < VEC; ++i) r.e[i] = blk[i].e[j];
    tile[ta * VEC + j][tb ^ ta] = r.v;
  }
  __syncthreads();
#pragma unroll
  for (int pass = 0; pass < VEC; ++pass) {
    const int r = pass * 16 + tb;
    const int64_t a = a0 + r, b = b0 + ta * VEC;
    if (a < p.sizeA && b < p.sizeB)
      *reinterpret_cast<uint4*>(out + out_off + a * p.out_strideA + b) = tile[r][ta ^ ((r / VEC) & 15)];
  }
}

// Scalar 32x32 tile transpose for extents that are not multiples of a vector.
template <typename T>
__global__ void __launch_bounds__(kThreads) transpose_tiled_scalar(const T* __restrict__ in, T* __restrict__ out,
                                                                   const TileParams p) {
  __shared__ T tile[32][33];
  uint32_t bid = blockIdx.x;   // tilesA * tilesB * batch = the grid size: every factor is below 2^32
  const uint32_t nA = static_cast<uint32_t>(p.tilesA), nB = static_cast<uint32_t>(p.tilesB);
  const uint32_t qA = bid / nA;
  const int64_t tileA = bid - qA * nA;
  bid = qA;
  const uint32_t qB = bid / nB;
  const int64_t tileB = bid - qB * nB;
  bid = qB;
  int64_t in_off, out_off;
  batch_offsets(p.batch, bid, in_off, out_off);
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t a0 = tileA * 32, b0 = tileB * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t b = b0 + ty + 8 * i, a = a0 + tx;
    if (a < p.sizeA && b < p.sizeB) tile[ty + 8 * i][tx] = in[in_off + b * p.in_strideB + a];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t a = a0 + ty + 8 * i, b = b0 + tx;
    if (a < p.sizeA && b < p.sizeB) out[out_off + a * p.out_strideA + b] = tile[tx][ty + 8 * i];
  }
}

struct GatherParams {   // generic strided gather, innermost output dim contiguous in the input too
  int n;                // dims, innermost last
  int64_t size[GL_MAX_DIMS];
  int64_t in_stride[GL_MAX_DIMS];
  int64_t total;        // number of VEC chunks
};

template <typename V, int ELEMS_PER_V>
__global__ void __launch_bounds__(kThreads) gather_rows(const V* __restrict__ in, V* __restrict__ out,
                                                        const GatherParams p) {
  // sizes and strides of the innermost dim are already counted in V units
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < p.total; c += (int64_t)gridDim.x * blockDim.x) {
    int64_t idx = c, off = 0;
#pragma unroll 1
    for (int d = p.n - 1; d >= 0; --d) {
      off += (idx % p.size[d]) * p.in_stride[d];
      idx /= p.size[d];
    }
    out[c] = in[off];
  }
}

template <typename T>
int run_transpose(const gl_ap* in, const int32_t* perm, gl_ap* out, cudaStream_t st) {
  constexpr int VEC = 16 / sizeof(T);
  // out dims with their input strides; drop size-1 dims, merge runs that stay adjacent
  int64_t istr_all[GL_MAX_DIMS];
  {
    int64_t s = 1;
    for (int d = in->ndim - 1; d >= 0; --d) { istr_all[d] = s; s *= in->shape[d]; }
  }
  int r = 0;
  int64_t size[GL_MAX_DIMS], istr[GL_MAX_DIMS];
  for (int j = 0; j < in->ndim; ++j) {
    const int64_t sz = in->shape[perm[j]], st_in = istr_all[perm[j]];
    if (sz == 1) continue;
    if (r > 0 && istr[r - 1] == st_in * sz) { size[r - 1] *= sz; istr[r - 1] = st_in; }
    else { size[r] = sz; istr[r] = st_in; ++r; }
  }
  const int64_t total = numel(*in);
  const T* src = static_cast<const T*>(in->data);
  T* dst = static_cast<T*>(out->data);
  if (r <= 1) {  // identity layout
    return cudaMemcpyAsync(dst, src, total * sizeof(T), cudaMemcpyDeviceToDevice, st) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  }
  int64_t ostr[GL_MAX_DIMS];
  {
    int64_t s = 1;
    for (int j = r - 1; j >= 0; --j) { ostr[j] = s; s *= size[j]; }
  }
  if (istr[r - 1] == 1) {  // innermost dim untouched: gather whole rows
    GatherParams g;
    std::memset(&g, 0, sizeof(g));
    g.n = r;
    const bool vec = size[r - 1] % VEC == 0;
    for (int j = 0; j < r; ++j) { g.size[j] = size[j]; g.in_stride[j] = vec ? istr[j] / VEC : istr[j]; }
    // (all outer input strides are multiples of the innermost extent, hence of VEC)
    if (vec) {
      g.size[r - 1] = size[r - 1] / VEC;
      g.in_stride[r - 1] = 1;
      g.total = total / VEC;
      gather_rows<uint4, VEC><<<grid_for(g.total, kThreads), kThreads, 0, st>>>(
          reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), g);
    } else {
      g.total = total;
      gather_rows<T, 1><<<grid_for(g.total, kThreads), kThreads, 0, st>>>(src, dst, g);
    }
    return launch_status();
  }
  // general case: tile over (A = the dim that is contiguous in the input, B = last output dim)
  int ja = -1;
  for (int j = 0; j < r; ++j) if (istr[j] == 1) ja = j;
  if (ja < 0) return GL_ERR_UNSUPPORTED;  // cannot happen for a dense input
  TileParams p;
  std::memset(&p, 0, sizeof(p));
  p.sizeA = size[ja];
  p.sizeB = size[r - 1];
  p.in_strideB = istr[r - 1];
  p.out_strideA = ostr[ja];
  int64_t nbatch = 1;
  for (int j = 0; j < r - 1; ++j) {
    if (j == ja) continue;
    const int k = p.batch.n++;
    p.batch.size[k] = size[j];
    p.batch.in_stride[k] = istr[j];
    p.batch.out_stride[k] = ostr[j];
    nbatch *= size[j];
  }
  const bool vec = p.sizeA % VEC == 0 && p.sizeB % VEC == 0;
  const int tile = vec ? 16 * VEC : 32;
  p.tilesA = (p.sizeA + tile - 1) / tile;
  p.tilesB = (p.sizeB + tile - 1) / tile;
  const int64_t blocks = p.tilesA * p.tilesB * nbatch;
  if (blocks > 0x7FFFFFFF) return GL_ERR_UNSUPPORTED;
  if (vec)
    return launch_pdl(transpose_tiled_vec<T, VEC>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, st, 1, src, dst,
                      p) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  else transpose_tiled_scalar<T><<<static_cast<unsigned>(blocks), kThreads, 0, st>>>(src, dst, p);
  return launch_status();
}

// ------------------------------------------------------------------------
// pad
// ------------------------------------------------------------------------

template <typename V>
__global__ void __launch_bounds__(kThreads) pad_kernel(const V* __restrict__ in, V* __restrict__ out, int64_t outer,
                                                       int64_t d_in, int64_t lo, int64_t d_out, int64_t inner,
                                                       V fill) {
  const int64_t total = outer * d_out * inner;
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < total; c += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = c % inner;
    const int64_t d = (c / inner) % d_out;
    const int64_t u = c / (inner * d_out);
    const int64_t s = d - lo;
    out[c] = (s >= 0 && s < d_in) ? in[(u * d_in + s) * inner + i] : fill;
  }
}

// pad of the innermost dimension, 4-byte elements, short rows: the output is walked as one flat array in
// 16-byte pieces (all lanes busy whatever the row length); the row of each element comes from one
// multiply-high division per piece and a carry test per element.
__global__ void __launch_bounds__(kThreads) pad_rows_flat(const uint32_t* __restrict__ in, uint32_t* __restrict__ out,
                                                          int64_t total, int d_in, int lo, int d_out, uint32_t mul,
                                                          uint32_t shift, uint32_t fill) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t pieces = total >> 2;
  for (int64_t pc = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; pc < pieces; pc += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t o = static_cast<uint32_t>(pc) << 2;         // total < 2^31
    uint32_t r = d_out == 1 ? o : (__umulhi(o, mul) >> shift);
    int c = static_cast<int>(o - r * static_cast<uint32_t>(d_out));
    // all four loads go out before the first select: border cells read a clamped address and are replaced
    uint32_t v[4];
    bool inside[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int x = c - lo;
      inside[i] = x >= 0 && x < d_in;
      v[i] = in[static_cast<int64_t>(r) * d_in + min(max(x, 0), d_in - 1)];
      if (++c == d_out) { c = 0; ++r; }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = inside[i] ? v[i] : fill;
    reinterpret_cast<uint4*>(out)[pc] = make_uint4(v[0], v[1], v[2], v[3]);
  }
  // the last total % 4 elements
  if (blockIdx.x == 0 && threadIdx.x < (total & 3)) {
    const int64_t o = (pieces << 2) + threadIdx.x;
    const int64_t r = o / d_out;
    const int x = static_cast<int>(o - r * d_out) - lo;
    out[o] = (x >= 0 && x < d_in) ? in[r * d_in + x] : fill;
  }
}

// pad of the innermost dimension: one warp per row, no divisions.
template <typename T>
__global__ void __launch_bounds__(kThreads) pad_rows(const T* __restrict__ in, T* __restrict__ out, int64_t rows,
                                                     int d_in, int lo, int d_out, T fill) {
  pdl_wait();
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  // a warp takes four rows per trip (rows r, r + warps, ...): four loads in flight per lane before any store
  for (int64_t r = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); r < rows; r += 4 * warps) {
    for (int x = lane; x < d_out; x += 32) {
      const bool inside = x >= lo && x < lo + d_in;
      T v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int64_t rr = r + j * warps;
        v[j] = fill;
        if (inside && rr < rows) v[j] = in[rr * d_in - lo + x];
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int64_t rr = r + j * warps;
        if (rr < rows) out[rr * d_out + x] = v[j];
      }
    }
  }
}

// ------------------------------------------------------------------------
// windows (materialised) and windows + reduceMax
// ------------------------------------------------------------------------

struct WinParams {
  int n;                          // compute dims
  int64_t in_size[GL_MAX_DIMS];   // b_i
  int64_t in_stride[GL_MAX_DIMS];
  int64_t out_ext[GL_MAX_DIMS];   // b'_i
  int64_t w[GL_MAX_DIMS], s[GL_MAX_DIMS], pad_lo[GL_MAX_DIMS];
  int64_t item;                   // elements of one input item
  int64_t wcells;                 // prod w_i
  int64_t total;                  // output elements
};

// General rank: one thread per output cell, out[a, p.., q..] = in[a, p_i s_i + q_i - pad_lo_i].
template <typename T>
__global__ void __launch_bounds__(kThreads) windows_generic(const T* __restrict__ in, T* __restrict__ out,
                                                            const WinParams p, T fill) {
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < p.total; c += (int64_t)gridDim.x * blockDim.x) {
    int64_t idx = c;
    int64_t q[GL_MAX_DIMS];
#pragma unroll 1
    for (int d = p.n - 1; d >= 0; --d) { q[d] = idx % p.w[d]; idx /= p.w[d]; }
    int64_t off = 0;
    bool inside = true;
#pragma unroll 1
    for (int d = p.n - 1; d >= 0; --d) {
      const int64_t pos = (idx % p.out_ext[d]) * p.s[d] + q[d] - p.pad_lo[d];
      idx /= p.out_ext[d];
      inside = inside && pos >= 0 && pos < p.in_size[d];
      off += pos * p.in_stride[d];
    }
    out[c] = inside ? in[idx * p.item + off] : fill;
  }
}

// General rank reduceMax over windows formed on the fly: one thread per window.
__global__ void __launch_bounds__(kThreads) window_max_generic(const float* __restrict__ in, float* __restrict__ out,
                                                               const WinParams p, int64_t nwin, float fill) {
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < nwin; c += (int64_t)gridDim.x * blockDim.x) {
    int64_t idx = c, base[GL_MAX_DIMS];
#pragma unroll 1
    for (int d = p.n - 1; d >= 0; --d) { base[d] = (idx % p.out_ext[d]) * p.s[d] - p.pad_lo[d]; idx /= p.out_ext[d]; }
    const float* item = in + idx * p.item;
    float best = -INFINITY;
#pragma unroll 1
    for (int64_t cell = 0; cell < p.wcells; ++cell) {
      int64_t cc = cell, off = 0;
      bool inside = true;
#pragma unroll 1
      for (int d = p.n - 1; d >= 0; --d) {
        const int64_t pos = base[d] + cc % p.w[d];
        cc /= p.w[d];
        inside = inside && pos >= 0 && pos < p.in_size[d];
        off += pos * p.in_stride[d];
      }
      best = fmaxf(best, inside ? item[off] : fill);
    }
    out[c] = best;
  }
}

// Convolution-style windows over ((N),(C,H,W)) items with window (C,Kh,Kw) and
// strides (1,Sh,Sw): the im2col matrix of Section 5.3, rows (n,h',w'), columns
// (c,kh,kw).  One block owns one (n,h'): it stages the Kh input rows of every
// channel in shared memory (border cells hold the fill value), then streams the
// Wo x K output slab, which is contiguous in memory, with 128-bit stores.
// Indexing is by warp (one staged row, then one output row per warp pass), so
// the inner loops carry no divisions; the staged row pitch is chosen on the host
// to spread the (c,kh,kw) gather over the shared-memory banks.
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void st_shared16(uint32_t smem_dst, const uint4& v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_last() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

struct Im2colParams {
  int64_t N, C, H, W, Kh, Kw, Sh, Sw, ph_lo, pw_lo, Ho, Wo, K;
  FastDiv by_Ho, by_Kh, by_Kw, by_border, by_segs, by_wv;   // divisors: Ho, Kh, Kw, border cells per row, segments per row, 16-byte pieces per input row
  int Cb, Kb;       // channels and columns per block (C / cparts, K / cparts)
  int lg, dc, dkh;  // aligned staging: 2^lg threads per row; channel and kernel-row step per pass
  int groups, segs; // sliding gather: 8-piece groups per row part, segments per output row
  int rsplit, gsplit;   // gsplit > 0: two phases; groups [0, gsplit) touch staged rows [0, rsplit) only
  int Wp;       // staged row length = W + pw_lo + pw_hi
  int pitch;    // staged row pitch in elements (>= Wp)
  int aligned;  // rows staged 16-byte aligned behind a margin of one 16-byte piece (W a multiple of it)
  int cparts;   // blocks per (n, h'): each takes C / cparts channels, i.e. K / cparts of the columns
  int slide;    // > 0: output columns per sliding-window item (4-byte elements, Sw = 1, Kw >= 3)
};

template <typename T, int VEC>
__global__ void __launch_bounds__(kThreads) im2col_rows(const T* __restrict__ in, T* __restrict__ out,
                                                        const Im2colParams p, T fill) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_wait();
  pdl_launch_dependents();
  // the grid is N * Ho * cparts blocks, below 2^31; this block owns channels [c0, c0 + Cb) = columns [k0, k0 + K)
  const unsigned part = blockIdx.x & static_cast<unsigned>(p.cparts - 1);   // cparts is 1 or 2
  const unsigned slab_id = blockIdx.x >> (p.cparts - 1);
  const unsigned n32 = fdiv(slab_id, p.by_Ho);
  const int64_t n = n32, ho = slab_id - n32 * static_cast<unsigned>(p.Ho);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int Cb = p.Cb, c0 = static_cast<int>(part) * Cb;
  const int Kw = static_cast<int>(p.Kw), Kh = static_cast<int>(p.Kh), rows = Cb * Kh;
  const int Kfull = static_cast<int>(p.K), K = p.Kb, k0 = static_cast<int>(part) * K;
  const int W = static_cast<int>(p.W), pw = static_cast<int>(p.pw_lo);
  int* lut = reinterpret_cast<int*>(smem_raw);                     // K entries: staged offset of column k at w'=0
  T* stage = reinterpret_cast<T*>(smem_raw + (((K + rows) * 4 + 15) / 16) * 16);   // [Cb*Kh][pitch]
  const int64_t h0 = ho * p.Sh - p.ph_lo;
  constexpr int LV = 16 / sizeof(T);   // elements per 16-byte piece
  if (p.aligned) {
    // Rows are 16-byte multiples and staged 16-byte aligned: cell w of a row sits at column LV + w, the
    // border cells left and right of it.  Every row piece is one asynchronous 16-byte copy, all of them
    // issued before the gather table is built, so the block waits for one round trip to L2 only.
    // The loop below is all 32-bit adds: row, channel and addresses advance incrementally.
    const int wv = W / LV;
    const int lg = p.lg;                              // 2^lg threads per staged row
    const int lpr = 1 << lg, rpp = blockDim.x >> lg;  // rows per pass
    const int li = threadIdx.x & (lpr - 1);
    const int H32 = static_cast<int>(p.H);
    const unsigned char* image = reinterpret_cast<const unsigned char*>(in + (n * p.C + c0) * p.H * p.W) + li * 16;
    union Vec { uint4 v; T e[LV]; };
    Vec fv;
#pragma unroll
    for (int e = 0; e < LV; ++e) fv.e[e] = fill;
    int r = threadIdx.x >> lg;
    int c = static_cast<int>(fdiv(r, p.by_Kh)), kh = r - c * Kh;
    const int dc = p.dc, dkh = p.dkh;                 // rows per pass = dc * Kh + dkh
    const int hbase = static_cast<int>(h0);
    const int rowbytes = W * static_cast<int>(sizeof(T));
    uint32_t sdst = static_cast<uint32_t>(__cvta_generic_to_shared(stage)) +
                    static_cast<uint32_t>((r * p.pitch + LV + li * LV) * static_cast<int>(sizeof(T)));
    const uint32_t sstep = static_cast<uint32_t>(rpp * p.pitch * static_cast<int>(sizeof(T)));
    auto stage_rows = [&](int limit) {
      for (; r < limit; r += rpp) {
        const int h = hbase + kh;
        const bool inside = static_cast<unsigned>(h) < static_cast<unsigned>(H32);
        const unsigned char* grow = image + static_cast<int64_t>(c * H32 + h) * rowbytes;   // C*H*W fits 31 bits
        for (int l = li, o = 0; l < wv; l += lpr, o += lpr * 16) {
          if (inside) cp_async16(sdst + o, grow + o);
          else st_shared16(sdst + o, fv.v);
        }
        kh += dkh; c += dc;
        if (kh >= Kh) { kh -= Kh; ++c; }
        sdst += sstep;
      }
    };
    // two copy groups when the gather below runs in two phases: rows [0, rsplit) first
    stage_rows(p.gsplit > 0 ? p.rsplit : rows);
    const int border = p.Wp - LV - W + pw;            // border cells per row: pw left, the rest right
    for (int e = threadIdx.x; e < rows * border; e += blockDim.x) {
      const int rr = static_cast<int>(fdiv(e, p.by_border)), j = e - rr * border;
      stage[rr * p.pitch + (j < pw ? LV - pw + j : LV + W + (j - pw))] = fill;
    }
    cp_async_commit();
    if (p.gsplit > 0) {
      stage_rows(rows);
      cp_async_commit();
    }
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
      const int row = static_cast<int>(fdiv(k, p.by_Kw));
      lut[k] = row * p.pitch + (k - row * Kw) + (LV - pw);
    }
    if (p.gsplit > 0) cp_async_wait_but_last();
    else cp_async_wait_all();
  } else if (p.W % LV == 0) {
    // Rows are 16-byte multiples, staged unaligned (any pitch, which matters for the 2-byte gather).
    // rowoff[r] = offset of staged row r inside this image, or -1 for a row of border cells; then every
    // thread takes 128-bit pieces of the flattened (row, piece) space, four loads in flight each.
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
      const int row = static_cast<int>(fdiv(k, p.by_Kw));
      lut[k] = row * p.pitch + (k - row * Kw);
    }
    int* rowoff = lut + K;   // the host reserves rows more ints behind the gather table
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
      const int c = static_cast<int>(fdiv(r, p.by_Kh)), kh = r - c * Kh;
      const int64_t h = h0 + kh;
      rowoff[r] = (h >= 0 && h < p.H) ? static_cast<int>((c * p.H + h) * p.W) : -1;
    }
    const int border = p.Wp - W;
    for (int e = threadIdx.x; e < rows * border; e += blockDim.x) {
      const int r = static_cast<int>(fdiv(e, p.by_border)), j = e - r * border;
      stage[r * p.pitch + (j < pw ? j : W + j)] = fill;
    }
    __syncthreads();
    const T* image = in + (n * p.C + c0) * p.H * p.W;
    const int wv = W / LV, slots = rows * wv;
    const FastDiv by_wv = p.by_wv;
    union Vec { uint4 v; T e[LV]; };
    for (int s0 = threadIdx.x; s0 < slots; s0 += 4 * blockDim.x) {
      Vec v[4];
      int at[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int sl = s0 + i * blockDim.x;
        at[i] = -1;
        if (sl < slots) {
          const int r = static_cast<int>(fdiv(sl, by_wv)), l = sl - r * wv;
          at[i] = r * p.pitch + pw + l * LV;
          const int off = rowoff[r];
          if (off >= 0) {
            v[i].v = *reinterpret_cast<const uint4*>(image + off + l * LV);
          } else {
#pragma unroll
            for (int e = 0; e < LV; ++e) v[i].e[e] = fill;
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (at[i] >= 0) {
#pragma unroll
          for (int e = 0; e < LV; ++e) stage[at[i] + e] = v[i].e[e];
        }
      }
    }
  } else {
    for (int k = threadIdx.x; k < K; k += blockDim.x) lut[k] = (k / Kw) * p.pitch + k % Kw;
    for (int r0 = warp * 4; r0 < rows; r0 += nwarps * 4) {
      for (int x = lane; x < p.Wp; x += 32) {
        const int w = x - pw;
        const bool col_ok = w >= 0 && w < W;
        T v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = r0 + i;
          const int c = r / Kh, kh = r - c * Kh;
          const int64_t h = h0 + kh;
          v[i] = (r < rows && col_ok && h >= 0 && h < p.H) ? in[((n * p.C + c0 + c) * p.H + h) * p.W + w] : fill;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (r0 + i < rows) stage[(r0 + i) * p.pitch + x] = v[i];
      }
    }
  }
  __syncthreads();
  T* slab = out + (n * p.Ho + ho) * p.Wo * p.K + k0;   // rows of Kfull columns, this block's start at k0
  const int Wo = static_cast<int>(p.Wo), Sw = static_cast<int>(p.Sw);
  union Chunk { uint4 v; T e[VEC]; };
  if (VEC == 4 && p.slide > 0) {
    // Sw = 1: the 16-byte piece (columns k..k+3) of output row w'+1 is the piece of row w' moved one
    // cell along its staged rows.  With Kw >= 3 a piece touches at most two staged rows, so a thread that
    // keeps its piece in registers and walks along w' reads two new cells per store instead of four.
    // Work items are (8 pieces, p.slide consecutive w'), one per quarter warp: every store of a quarter is
    // one whole 128-byte line.  Neighbouring quarters take neighbouring segments; with an odd segment
    // length their staged columns differ modulo 4, which keeps them on different shared-memory banks
    // (rows start on 16-byte boundaries, so one column of different rows covers eight banks only).
    const int L = p.slide, ppr = K / 4, groups = p.groups, segs = p.segs;
    const int qi = threadIdx.x >> 3, nq = blockDim.x >> 3, ql = threadIdx.x & 7;
    int item = qi;
    auto run_items = [&](int limit) {
      for (; item < limit; item += nq) {
        const int g = static_cast<int>(fdiv(item, p.by_segs)), seg = item - g * segs;
        const int piece = g * 8 + ql;
        if (piece >= ppr) continue;
        const int k = piece * 4, wo0 = seg * L, cnt = min(L, Wo - wo0);
        const int4 a = *reinterpret_cast<const int4*>(lut + k);
        const int la = a.y != a.x + 1 ? 1 : a.z != a.y + 1 ? 2 : a.w != a.z + 1 ? 3 : 4;   // cells in the first staged row
        const T* srcA = stage + (la == 1 ? a.x : la == 2 ? a.y : la == 3 ? a.z : a.w) + wo0;
        const T* srcB = stage + a.w + wo0;
        T* o = slab + static_cast<int64_t>(wo0) * Kfull + k;
        Chunk ch;
        ch.e[0] = stage[a.x + wo0]; ch.e[1] = stage[a.y + wo0]; ch.e[2] = stage[a.z + wo0]; ch.e[3] = stage[a.w + wo0];
        *reinterpret_cast<uint4*>(o) = ch.v;
        for (int j = 1; j < cnt; ++j) {
          const T na = srcA[j], nb = srcB[j];
          ch.e[0] = la == 1 ? na : ch.e[1];
          ch.e[1] = la == 2 ? na : ch.e[2];
          ch.e[2] = la == 3 ? na : ch.e[3];
          ch.e[3] = la == 4 ? na : nb;
          o += Kfull;
          *reinterpret_cast<uint4*>(o) = ch.v;
        }
      }
    };
    if (p.gsplit > 0) {
      // the first gsplit groups read staged rows below rsplit only: they are written while the second
      // copy group is still in flight
      run_items(p.gsplit * segs);
      cp_async_wait_all();
      __syncthreads();
    }
    run_items(groups * segs);
    return;
  }
  constexpr int kLutPasses = 5;
  int lutreg[kLutPasses][VEC];
  if (VEC > 1 && K <= kLutPasses * 32 * VEC) {
#pragma unroll
    for (int t = 0; t < kLutPasses; ++t)
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        const int k = (t * 32 + lane) * VEC + i;
        lutreg[t][i] = k < K ? lut[k] : 0;
      }
  }
  for (int wo = warp; wo < Wo; wo += nwarps) {
    const T* base = stage + wo * Sw;
    T* orow = slab + static_cast<int64_t>(wo) * Kfull;
    if (VEC == 1) {
      for (int k = lane; k < K; k += 32) orow[k] = base[lut[k]];
    } else if (K <= kLutPasses * 32 * VEC) {
      // the gather offsets of this lane do not depend on the output row: keep them in registers
#pragma unroll
      for (int t = 0; t < kLutPasses; ++t) {
        const int k = (t * 32 + lane) * VEC;
        if (k < K) {
          Chunk ch;
#pragma unroll
          for (int i = 0; i < VEC; ++i) ch.e[i] = base[lutreg[t][i]];
          *reinterpret_cast<uint4*>(orow + k) = ch.v;
        }
      }
    } else {
      for (int k = lane * VEC; k < K; k += 32 * VEC) {
        Chunk ch;
#pragma unroll
        for (int i = 0; i < VEC; ++i) ch.e[i] = base[lut[k + i]];
        *reinterpret_cast<uint4*>(orow + k) = ch.v;
      }
    }
  }
}

// Row pitch (>= Wp, < Wp + 32) with the fewest shared-memory bank conflicts for the
// gather "lane reads staged[(k/Kw)*pitch + k%Kw], k = VEC*lane + i" (4-byte banks).
int best_im2col_pitch(int Wp, int Kw, int K, int vec, int elem_bytes, int step = 1) {
  const int first = (Wp + step - 1) / step * step;   // pitches are multiples of step
  int best = first, best_cost = 1 << 30;
  for (int pitch = first; pitch < first + 32; pitch += step) {
    int cost = 0;
    for (int pass = 0; pass * 32 * vec < K && pass < 8; ++pass)
      for (int i = 0; i < vec; ++i) {
        int hits[32] = {0}, worst = 0;
        for (int lane = 0; lane < 32; ++lane) {
          const int k = pass * 32 * vec + lane * vec + i;
          if (k >= K) break;
          const int bank = (((k / Kw) * pitch + k % Kw) * elem_bytes / 4) & 31;
          worst = std::max(worst, ++hits[bank]);
        }
        cost += worst;
      }
    if (cost < best_cost) { best_cost = cost; best = pitch; }
  }
  return best;
}

// 2D windows + reduceMax over ((..),(H,W)) items (Fig. 2c): one thread per output.
__global__ void __launch_bounds__(kThreads) window_max_2d(const float* __restrict__ in, float* __restrict__ out,
                                                           int64_t planes, int H, int W, int Kh, int Kw, int Sh, int Sw,
                                                           int ph, int pw, int Ho, int Wo, float fill) {
  const int64_t total = planes * Ho * Wo;
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < total; c += (int64_t)gridDim.x * blockDim.x) {
    const int y = static_cast<int>(c % Wo);
    const int x = static_cast<int>((c / Wo) % Ho);
    const float* plane = in + (c / ((int64_t)Wo * Ho)) * H * W;
    float best = -INFINITY;
    for (int dx = 0; dx < Kh; ++dx) {
      const int h = x * Sh + dx - ph;
      for (int dy = 0; dy < Kw; ++dy) {
        const int w = y * Sw + dy - pw;
        const bool inside = h >= 0 && h < H && w >= 0 && w < W;
        best = fmaxf(best, inside ? plane[(int64_t)h * W + w] : fill);
      }
    }
    out[c] = best;
  }
}

// The same for 2-byte (bf16) planes: values are compared as floats (every bf16 value is a float, and the
// largest of them is one of them, so nothing is rounded).
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

__global__ void __launch_bounds__(kThreads) window_max_2d_bf16(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                                                int64_t planes, int H, int W, int Kh, int Kw, int Sh, int Sw,
                                                                int ph, int pw, int Ho, int Wo, float fill) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t total = planes * Ho * Wo;
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < total; c += (int64_t)gridDim.x * blockDim.x) {
    const int y = static_cast<int>(c % Wo);
    const int x = static_cast<int>((c / Wo) % Ho);
    const uint16_t* plane = in + (c / ((int64_t)Wo * Ho)) * H * W;
    float best = -INFINITY;
    for (int dx = 0; dx < Kh; ++dx) {
      const int h = x * Sh + dx - ph;
      for (int dy = 0; dy < Kw; ++dy) {
        const int w = y * Sw + dy - pw;
        const bool inside = h >= 0 && h < H && w >= 0 && w < W;
        best = fmaxf(best, inside ? bf16_bits_to_float(plane[(int64_t)h * W + w]) : fill);
      }
    }
    out[c] = static_cast<uint16_t>(__float_as_uint(best) >> 16);
  }
}

// Channels-last items: compute reduceMax (windows (access act 1) (Kh,Kw,1) (Sh,Sw,1)) on ((N),(H,W,C)), the max
// pooling of Fig. 2c with the channel as the innermost dimension.  A thread owns one output pixel and one
// 16-byte piece of its channels (4 floats or 8 bf16 values): every load is a full piece, consecutive threads
// read consecutive pieces.  Border cells count as `fill`.
struct PoolHwc {
  int H, W, Kh, Kw, Sh, Sw, ph, pw, Ho, Wo, cv;   // cv: 16-byte pieces per pixel
  int split_log2;                                 // 2^split_log2 neighbouring lanes share one output piece
  int64_t total;                                  // N * Ho * Wo * cv << split_log2
  FastDiv by_cv, by_Wo, by_Ho, by_Kw;
};

// Large windows over few outputs (a pooling layer that ends a network) would leave most of the machine idle with
// one thread per output piece, so 2^split_log2 neighbouring lanes share a piece: lane j takes the window cells
// j, j + 2^split_log2, ... and the lanes' maxima are combined by shuffles.
template <bool BF16>
__global__ void __launch_bounds__(kThreads) window_max_hwc(const uint4* __restrict__ in, uint4* __restrict__ out, const PoolHwc p,
                                                            float fill) {
  pdl_wait();
  pdl_launch_dependents();
  const int split = 1 << p.split_log2, taps = p.Kh * p.Kw;
  // all threads of a warp take part in the shuffles: the loop bound is rounded up to whole blocks
  const int64_t total_r = (p.total + blockDim.x - 1) / blockDim.x * blockDim.x;
  for (int64_t e0 = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e0 < total_r; e0 += (int64_t)gridDim.x * blockDim.x) {
    const bool live = e0 < p.total;
    const uint32_t e = static_cast<uint32_t>(live ? e0 : 0) >> p.split_log2, part = static_cast<uint32_t>(e0) & (split - 1);
    uint32_t pix, v, row, wo, n, ho;
    p.by_cv.divmod(e, pix, v);
    p.by_Wo.divmod(pix, row, wo);
    p.by_Ho.divmod(row, n, ho);
    float best[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) best[i] = -INFINITY;
    bool border = false;
    const uint4* img = in + static_cast<int64_t>(n) * p.H * p.W * p.cv + v;
#pragma unroll 4
    for (int t = part; t < taps; t += split) {
      uint32_t dy, dx;
      p.by_Kw.divmod(static_cast<uint32_t>(t), dy, dx);
      const int h = static_cast<int>(ho) * p.Sh + static_cast<int>(dy) - p.ph;
      const int w = static_cast<int>(wo) * p.Sw + static_cast<int>(dx) - p.pw;
      if (h < 0 || h >= p.H || w < 0 || w >= p.W) { border = true; continue; }
      const uint4 q = img[(static_cast<int64_t>(h) * p.W + w) * p.cv];
      const uint32_t qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (BF16) {
          best[2 * i] = fmaxf(best[2 * i], bf16_bits_to_float(qq[i] & 0xFFFFu));
          best[2 * i + 1] = fmaxf(best[2 * i + 1], __uint_as_float(qq[i] & 0xFFFF0000u));
        } else {
          best[i] = fmaxf(best[i], __uint_as_float(qq[i]));
        }
      }
    }
    if (border) {
#pragma unroll
      for (int i = 0; i < 8; ++i) best[i] = fmaxf(best[i], fill);
    }
    for (int d = 1; d < split; d <<= 1) {
#pragma unroll
      for (int i = 0; i < 8; ++i) best[i] = fmaxf(best[i], __shfl_xor_sync(0xffffffffu, best[i], d));
    }
    if (live && part == 0) {
      uint4 r;
      if (BF16) {
        r.x = (__float_as_uint(best[0]) >> 16) | (__float_as_uint(best[1]) & 0xFFFF0000u);
        r.y = (__float_as_uint(best[2]) >> 16) | (__float_as_uint(best[3]) & 0xFFFF0000u);
        r.z = (__float_as_uint(best[4]) >> 16) | (__float_as_uint(best[5]) & 0xFFFF0000u);
        r.w = (__float_as_uint(best[6]) >> 16) | (__float_as_uint(best[7]) & 0xFFFF0000u);
      } else {
        r = make_uint4(__float_as_uint(best[0]), __float_as_uint(best[1]), __float_as_uint(best[2]), __float_as_uint(best[3]));
      }
      out[e] = r;
    }
  }
}

// The same with the window shape fixed at compile time: all KH*KW pieces are requested before the first maximum
// is taken (addresses of border cells are clamped into the image and their values replaced by `fill`), so a
// thread has KH*KW loads in flight instead of one chain of load, compare, next address.
template <bool BF16, int KH, int KW>
__global__ void __launch_bounds__(kThreads) window_max_hwc_fixed(const uint4* __restrict__ in, uint4* __restrict__ out,
                                                                  const PoolHwc p, float fill) {
  const int64_t e0 = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const bool live = e0 < p.total;
  uint32_t pix, v, row, wo, n, ho;
  p.by_cv.divmod(static_cast<uint32_t>(live ? e0 : 0), pix, v);
  p.by_Wo.divmod(pix, row, wo);
  p.by_Ho.divmod(row, n, ho);
  const uint4* img = in + static_cast<int64_t>(n) * p.H * p.W * p.cv + v;
  pdl_wait();
  pdl_launch_dependents();
  if (!live) return;
  uint4 q[KH * KW];
  bool inside[KH * KW];
#pragma unroll
  for (int dy = 0; dy < KH; ++dy) {
#pragma unroll
    for (int dx = 0; dx < KW; ++dx) {
      const int h = static_cast<int>(ho) * p.Sh + dy - p.ph, w = static_cast<int>(wo) * p.Sw + dx - p.pw;
      inside[dy * KW + dx] = h >= 0 && h < p.H && w >= 0 && w < p.W;
      const int hc = min(max(h, 0), p.H - 1), wc = min(max(w, 0), p.W - 1);
      q[dy * KW + dx] = img[(static_cast<int64_t>(hc) * p.W + wc) * p.cv];
    }
  }
  float best[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) best[i] = -INFINITY;
#pragma unroll
  for (int t = 0; t < KH * KW; ++t) {
    const uint32_t qq[4] = {q[t].x, q[t].y, q[t].z, q[t].w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (BF16) {
        best[2 * i] = fmaxf(best[2 * i], inside[t] ? bf16_bits_to_float(qq[i] & 0xFFFFu) : fill);
        best[2 * i + 1] = fmaxf(best[2 * i + 1], inside[t] ? __uint_as_float(qq[i] & 0xFFFF0000u) : fill);
      } else {
        best[i] = fmaxf(best[i], inside[t] ? __uint_as_float(qq[i]) : fill);
      }
    }
  }
  uint4 r;
  if (BF16) {
    r.x = (__float_as_uint(best[0]) >> 16) | (__float_as_uint(best[1]) & 0xFFFF0000u);
    r.y = (__float_as_uint(best[2]) >> 16) | (__float_as_uint(best[3]) & 0xFFFF0000u);
    r.z = (__float_as_uint(best[4]) >> 16) | (__float_as_uint(best[5]) & 0xFFFF0000u);
    r.w = (__float_as_uint(best[6]) >> 16) | (__float_as_uint(best[7]) & 0xFFFF0000u);
  } else {
    r = make_uint4(__float_as_uint(best[0]), __float_as_uint(best[1]), __float_as_uint(best[2]), __float_as_uint(best[3]));
  }
  out[e0] = r;
}

// 2D windows + reduceMax, tiled: one block owns TH output rows of one plane.  It
// stages the (TH-1)*Sh+Kh input rows it needs (border cells hold the fill value)
// with 128-bit loads, then every thread reduces whole windows out of shared
// memory.  Each input cell is read from HBM once per block.
struct PoolTile {
  int H, W, Kh, Kw, Sh, Sw, ph, pw, Ho, Wo;
  int TH;        // output rows per block
  int tiles;     // row tiles per plane
  int Wp;        // staged row length = pw + W + right border
  int vec;       // rows are 16-byte multiples: float4 loads
};

// T: float, or uint16_t for bf16 planes (staged and compared as floats; the largest value is one of the inputs, so
// storing its upper 16 bits rounds nothing).  `vec` rows are read as 16-byte pieces: 4 floats or 8 bf16 values.
__device__ __forceinline__ float pool_load(const float* p) { return *p; }
__device__ __forceinline__ float pool_load(const uint16_t* p) { return bf16_bits_to_float(*p); }
__device__ __forceinline__ void pool_store(float* p, float v) { *p = v; }
__device__ __forceinline__ void pool_store(uint16_t* p, float v) { *p = static_cast<uint16_t>(__float_as_uint(v) >> 16); }

template <typename T>
__global__ void __launch_bounds__(kThreads) window_max_2d_tiled(const T* __restrict__ in, T* __restrict__ out,
                                                                 const PoolTile p, float fill) {
  extern __shared__ __align__(16) float pool_stage[];
  constexpr int kPer = 16 / static_cast<int>(sizeof(T));   // elements per 16-byte piece
  const int64_t plane = blockIdx.x / p.tiles;
  const int tile = blockIdx.x % p.tiles;
  const int y0 = tile * p.TH;
  const int th = min(p.TH, p.Ho - y0);
  const int rows = (th - 1) * p.Sh + p.Kh;
  const int h0 = y0 * p.Sh - p.ph;
  const T* src = in + plane * p.H * p.W;
  // left and right border columns, then the rows themselves
  const int right = p.Wp - p.pw - p.W;
  for (int e = threadIdx.x; e < rows * (p.pw + right); e += blockDim.x) {
    const int r = e / (p.pw + right), j = e % (p.pw + right);
    pool_stage[r * p.Wp + (j < p.pw ? j : p.W + j)] = fill;
  }
  if (p.vec) {
    const int wv = p.W / kPer;
    for (int e = threadIdx.x; e < rows * wv; e += blockDim.x) {
      const int r = e / wv, x = (e - r * wv) * kPer;
      const int h = h0 + r;
      float* d = pool_stage + r * p.Wp + p.pw + x;
      if (h >= 0 && h < p.H) {
        const uint4 q = *reinterpret_cast<const uint4*>(src + (int64_t)h * p.W + x);
        const uint32_t qq[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (kPer == 4) d[i] = __uint_as_float(qq[i]);
          else { d[2 * i] = bf16_bits_to_float(qq[i] & 0xFFFFu); d[2 * i + 1] = __uint_as_float(qq[i] & 0xFFFF0000u); }
        }
      } else {
#pragma unroll
        for (int i = 0; i < kPer; ++i) d[i] = fill;
      }
    }
  } else {
    for (int e = threadIdx.x; e < rows * p.W; e += blockDim.x) {
      const int r = e / p.W, x = e - r * p.W;
      const int h = h0 + r;
      pool_stage[r * p.Wp + p.pw + x] = (h >= 0 && h < p.H) ? pool_load(src + (int64_t)h * p.W + x) : fill;
    }
  }
  __syncthreads();
  T* dst = out + (plane * p.Ho + y0) * p.Wo;
  for (int e = threadIdx.x; e < th * p.Wo; e += blockDim.x) {
    const int y = e / p.Wo, x = e - y * p.Wo;
    const float* win = pool_stage + (y * p.Sh) * p.Wp + x * p.Sw;
    float best = -INFINITY;
    for (int dy = 0; dy < p.Kh; ++dy)
      for (int dx = 0; dx < p.Kw; ++dx) best = fmaxf(best, win[dy * p.Wp + dx]);
    pool_store(dst + e, best);
  }
}

// Tiling of window_max_2d_tiled: as many output rows per block as fit 24 KB of staged floats.
inline bool plan_pool_tile(const gl_ap* in, const gl_windows* w, const gl_ap& A, int na, int per_piece, PoolTile* t) {
  t->H = (int)in->shape[na]; t->W = (int)in->shape[na + 1];
  t->Kh = (int)w->wshape[0]; t->Kw = (int)w->wshape[1];
  t->Sh = (int)w->stride[0]; t->Sw = (int)w->stride[1];
  t->ph = (int)w->pad_lo[0]; t->pw = (int)w->pad_lo[1];
  t->Ho = (int)A.shape[na]; t->Wo = (int)A.shape[na + 1];
  // staged columns: left border, the row, and whatever the last window reaches beyond it
  t->Wp = std::max(t->pw + t->W, (t->Wo - 1) * t->Sw + t->Kw);
  t->vec = (t->W % per_piece == 0) ? 1 : 0;
  const int budget = 24 * 1024 / 4;   // floats of shared memory per block
  const int max_rows = budget / t->Wp;
  if (max_rows < t->Kh) return false;
  t->TH = std::min(t->Ho, (max_rows - t->Kh) / t->Sh + 1);
  t->tiles = (t->Ho + t->TH - 1) / t->TH;
  t->TH = (t->Ho + t->tiles - 1) / t->tiles;   // even out the tiles
  return prod(in->shape, 0, na) * t->tiles <= 0x7FFFFFFF;
}

// Fig. 2c with a 3x3 window, stride 2 and one border cell on the low side (the pooling layer of
// ResNet-style networks), rows that are multiples of four floats: no staging at all.  A thread
// owns four input columns (two outputs) and walks R output rows downwards; each input row is read
// once with one 128-bit load plus the neighbour's last column, its two horizontal maxima are kept
// in registers, and the odd rows are shared by two consecutive output rows.
struct Pool3s2 {
  int H, W, Ho, Wo, R, strips, w4;
  int64_t units;   // planes * strips
  FastDiv by_strips;   // used when units < 2^31
};

template <int R>
__global__ void __launch_bounds__(256) window_max_3x3s2(const float* __restrict__ in, float* __restrict__ out,
                                                         const Pool3s2 p, float fill) {
  pdl_wait();
  pdl_launch_dependents();
  const int64_t u = blockIdx.x * (int64_t)blockDim.y + threadIdx.y;
  if (u >= p.units) return;
  const int64_t plane = p.units < (1ll << 31) ? static_cast<int64_t>(fdiv(static_cast<uint32_t>(u), p.by_strips)) : u / p.strips;
  const int strip = static_cast<int>(u - plane * p.strips);
  const float* src = in + plane * p.H * p.W;
  float* dst = out + plane * p.Ho * p.Wo;
  const int y0 = strip * R;
  for (int j = threadIdx.x; j < p.w4; j += blockDim.x) {
    // all 2R+1 input rows of the strip are requested before the first maximum is taken
    float4 v[2 * R + 1];
    float left[2 * R + 1];
#pragma unroll
    for (int i = 0; i < 2 * R + 1; ++i) {
      const int h = 2 * y0 - 1 + i;
      if (h >= 0 && h < p.H) {
        const float* row = src + (int64_t)h * p.W + 4 * j;
        v[i] = *reinterpret_cast<const float4*>(row);
        left[i] = j > 0 ? row[-1] : fill;
      } else {
        v[i] = make_float4(fill, fill, fill, fill);
        left[i] = fill;
      }
    }
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int y = y0 + i;
      if (y < p.Ho) {
        float o0 = -INFINITY, o1 = -INFINITY;
#pragma unroll
        for (int d = 0; d < 3; ++d) {
          const float4 w = v[2 * i + d];
          o0 = fmaxf(o0, fmaxf(fmaxf(left[2 * i + d], w.x), w.y));
          o1 = fmaxf(o1, fmaxf(fmaxf(w.y, w.z), w.w));
        }
        *reinterpret_cast<float2*>(dst + (int64_t)y * p.Wo + 2 * j) = make_float2(o0, o1);
      }
    }
  }
}

// The same with the (plane, strip, column group) items dealt to threads one by one, so that every lane of a warp
// has work whatever the row length (rows of 28 column groups leave four lanes of a warp-per-strip layout idle).
template <int R>
__global__ void __launch_bounds__(256) window_max_3x3s2_flat(const float* __restrict__ in, float* __restrict__ out,
                                                              const Pool3s2 p, int64_t items, FastDiv by_w4, float fill) {
  const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const bool live = t < items;
  uint32_t rest, j, plane, strip;
  by_w4.divmod(static_cast<uint32_t>(live ? t : 0), rest, j);
  p.by_strips.divmod(rest, plane, strip);
  const float* src = in + static_cast<int64_t>(plane) * p.H * p.W;
  float* dst = out + static_cast<int64_t>(plane) * p.Ho * p.Wo;
  const int y0 = static_cast<int>(strip) * R;
  pdl_wait();
  pdl_launch_dependents();
  if (!live) return;
  float4 v[2 * R + 1];
  float left[2 * R + 1];
#pragma unroll
  for (int i = 0; i < 2 * R + 1; ++i) {
    const int h = 2 * y0 - 1 + i;
    if (h >= 0 && h < p.H) {
      const float* row = src + (int64_t)h * p.W + 4 * j;
      v[i] = *reinterpret_cast<const float4*>(row);
      left[i] = j > 0 ? row[-1] : fill;
    } else {
      v[i] = make_float4(fill, fill, fill, fill);
      left[i] = fill;
    }
  }
#pragma unroll
  for (int i = 0; i < R; ++i) {
    const int y = y0 + i;
    if (y < p.Ho) {
      float o0 = -INFINITY, o1 = -INFINITY;
#pragma unroll
      for (int d = 0; d < 3; ++d) {
        const float4 w = v[2 * i + d];
        o0 = fmaxf(o0, fmaxf(fmaxf(left[2 * i + d], w.x), w.y));
        o1 = fmaxf(o1, fmaxf(fmaxf(w.y, w.z), w.w));
      }
      *reinterpret_cast<float2*>(dst + (int64_t)y * p.Wo + 2 * j) = make_float2(o0, o1);
    }
  }
}

// The same pooling on 2-byte planes (rows that are multiples of eight values): a thread owns eight input
// columns (four outputs) of one strip of R output rows.  bf16 values are compared as the floats they stand for
// (a shift), so the maximum is exact.
struct Pool3s2H {
  int H, W, Ho, Wo, strips, w8;
  int64_t items;   // planes * strips * w8
  FastDiv by_w8, by_strips;
};

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t bf16_pack_exact(float lo, float hi) {   // both already bf16 values
  return (__float_as_uint(lo) >> 16) | (__float_as_uint(hi) & 0xFFFF0000u);
}

template <int R>
__global__ void __launch_bounds__(256) window_max_3x3s2_bf16(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                                              const Pool3s2H p, float fill) {
  const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (t >= p.items) { pdl_wait(); pdl_launch_dependents(); return; }
  uint32_t rest, j, plane, strip;
  p.by_w8.divmod(static_cast<uint32_t>(t), rest, j);
  p.by_strips.divmod(rest, plane, strip);
  const uint16_t* src = in + static_cast<int64_t>(plane) * p.H * p.W;
  uint16_t* dst = out + static_cast<int64_t>(plane) * p.Ho * p.Wo;
  const int y0 = static_cast<int>(strip) * R;
  pdl_wait();
  pdl_launch_dependents();
  uint4 v[2 * R + 1];
  float left[2 * R + 1];
  const uint32_t fill2 = bf16_pack_exact(fill, fill);
#pragma unroll
  for (int i = 0; i < 2 * R + 1; ++i) {
    const int h = 2 * y0 - 1 + i;
    if (h >= 0 && h < p.H) {
      const uint16_t* row = src + (int64_t)h * p.W + 8 * j;
      v[i] = *reinterpret_cast<const uint4*>(row);
      left[i] = j > 0 ? bf16_lo(row[-1]) : fill;
    } else {
      v[i] = make_uint4(fill2, fill2, fill2, fill2);
      left[i] = fill;
    }
  }
#pragma unroll
  for (int i = 0; i < R; ++i) {
    const int y = y0 + i;
    if (y < p.Ho) {
      float o0 = -INFINITY, o1 = -INFINITY, o2 = -INFINITY, o3 = -INFINITY;
#pragma unroll
      for (int d = 0; d < 3; ++d) {
        const uint4 w = v[2 * i + d];
        const float x1 = bf16_hi(w.x), x3 = bf16_hi(w.y), x5 = bf16_hi(w.z);
        o0 = fmaxf(o0, fmaxf(fmaxf(left[2 * i + d], bf16_lo(w.x)), x1));
        o1 = fmaxf(o1, fmaxf(fmaxf(x1, bf16_lo(w.y)), x3));
        o2 = fmaxf(o2, fmaxf(fmaxf(x3, bf16_lo(w.z)), x5));
        o3 = fmaxf(o3, fmaxf(fmaxf(x5, bf16_lo(w.w)), bf16_hi(w.w)));
      }
      *reinterpret_cast<uint2*>(dst + (int64_t)y * p.Wo + 4 * j) = make_uint2(bf16_pack_exact(o0, o1), bf16_pack_exact(o2, o3));
    }
  }
}

// 2-byte planes whose windows are eight columns wide, eight apart and unpadded in W (rows of a multiple of
// eight values): every window row is one aligned 16-byte piece.  A thread owns one window; its Kh pieces are
// requested eight at a time (rows outside the plane: address clamped, value replaced by `fill`).
struct PoolRow8 {
  int H, W, Kh, Sh, ph, Ho, Wo;
  int64_t total;   // planes * Ho * Wo
  FastDiv by_Wo, by_Ho;
};

__global__ void __launch_bounds__(kThreads) window_max_rows8_bf16(const uint16_t* __restrict__ in, uint16_t* __restrict__ out,
                                                                   const PoolRow8 p, float fill) {
  const int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const bool live = e < p.total;
  uint32_t row, wo, plane, ho;
  p.by_Wo.divmod(static_cast<uint32_t>(live ? e : 0), row, wo);
  p.by_Ho.divmod(row, plane, ho);
  const uint16_t* src = in + static_cast<int64_t>(plane) * p.H * p.W + 8 * wo;
  pdl_wait();
  pdl_launch_dependents();
  if (!live) return;
  float best = -INFINITY;
  const int h0 = static_cast<int>(ho) * p.Sh - p.ph;
  for (int d0 = 0; d0 < p.Kh; d0 += 8) {
    uint4 q[8];
#pragma unroll
    for (int d = 0; d < 8; ++d) {
      const int h = min(max(h0 + d0 + d, 0), p.H - 1);
      q[d] = *reinterpret_cast<const uint4*>(src + static_cast<int64_t>(h) * p.W);
    }
#pragma unroll
    for (int d = 0; d < 8; ++d) {
      const int h = h0 + d0 + d;
      if (d0 + d < p.Kh) {
        float m = fill;
        if (h >= 0 && h < p.H) {
          m = fmaxf(fmaxf(fmaxf(bf16_lo(q[d].x), bf16_hi(q[d].x)), fmaxf(bf16_lo(q[d].y), bf16_hi(q[d].y))),
                    fmaxf(fmaxf(bf16_lo(q[d].z), bf16_hi(q[d].z)), fmaxf(bf16_lo(q[d].w), bf16_hi(q[d].w))));
        }
        best = fmaxf(best, m);
      }
    }
  }
  out[e] = static_cast<uint16_t>(__float_as_uint(best) >> 16);
}

// reduceMax of whole items (no windows): one warp per item.
__global__ void __launch_bounds__(kThreads) item_max(const float* __restrict__ in, float* __restrict__ out,
                                                      int64_t items, int64_t item) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t a = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); a < items; a += warps) {
    float best = -INFINITY;
    for (int64_t i = lane; i < item; i += 32) best = fmaxf(best, in[a * item + i]);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) best = fmaxf(best, __shfl_xor_sync(0xFFFFFFFFu, best, s));
    if (lane == 0) out[a] = best;
  }
}

__global__ void __launch_bounds__(kThreads) relu_vec(const float4* __restrict__ in, float4* __restrict__ out, int64_t n4) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  // while the predecessor drains, the lines of this thread's first trip are requested into L2 (a prefetch consumes
  // nothing; a line the predecessor still writes is updated in L2, where all writes meet)
  {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (i + j * stride < n4) asm volatile("prefetch.global.L2 [%0];" ::"l"(in + i + j * stride) : "memory");
  }
  pdl_wait();
  pdl_launch_dependents();
  // four independent 16-byte loads in flight per thread
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += 4 * stride) {
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (i + j * stride < n4) v[j] = in[i + j * stride];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (i + j * stride < n4) {
        float4 r = v[j];
        r.x = r.x > 0.f ? r.x : 0.f;
        r.y = r.y > 0.f ? r.y : 0.f;
        r.z = r.z > 0.f ? r.z : 0.f;
        r.w = r.w > 0.f ? r.w : 0.f;
        out[i + j * stride] = r;
      }
  }
}

__global__ void relu_tail(const float* __restrict__ in, float* __restrict__ out, int64_t from, int64_t n) {
  const int64_t i = from + threadIdx.x;
  if (i < n) out[i] = in[i] > 0.f ? in[i] : 0.f;
}

// slice / concat / pair: dst[u, dst_off + d, i] = src[u, src_off + d, i] for d < count, the tensors seen
// as (outer, dim, inner).
template <typename V>
__global__ void __launch_bounds__(kThreads) copy_dim_block(const V* __restrict__ src, V* __restrict__ dst,
                                                           int64_t outer, int64_t d_src, int64_t src_off,
                                                           int64_t d_dst, int64_t dst_off, int64_t count,
                                                           int64_t inner) {
  const int64_t total = outer * count * inner;
  for (int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; c < total; c += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = c % inner;
    const int64_t d = (c / inner) % count;
    const int64_t u = c / (inner * count);
    dst[(u * d_dst + dst_off + d) * inner + i] = src[(u * d_src + src_off + d) * inner + i];
  }
}

// reduceSum of whole items: one warp per item, lane l adds cells l, l+32, ... in order, then a
// fixed butterfly: the order of additions does not depend on the launch.
__global__ void __launch_bounds__(kThreads) item_sum(const float* __restrict__ in, float* __restrict__ out,
                                                      int64_t items, int64_t item) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t a = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); a < items; a += warps) {
    float acc = 0.f;
    for (int64_t i = lane; i < item; i += 32) acc += in[a * item + i];
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, s);
    if (lane == 0) out[a] = acc;
  }
}

int run_copy_dim(const void* src, void* dst, int dtype, int64_t outer, int64_t d_src, int64_t src_off, int64_t d_dst,
                 int64_t dst_off, int64_t count, int64_t inner, cudaStream_t st) {
  const size_t es = dtype_size(dtype);
  const int vec = static_cast<int>(16 / es);
  const int64_t total = outer * count * inner;
  if (total == 0) return GL_OK;
  if (inner % vec == 0) {   // every row piece starts on a 16-byte boundary (bases are 16-byte aligned)
    const int64_t iv = inner / vec;
    copy_dim_block<uint4><<<grid_for(outer * count * iv, kThreads), kThreads, 0, st>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), outer, d_src, src_off, d_dst, dst_off, count, iv);
  } else if (dtype == GL_F32) {
    copy_dim_block<uint32_t><<<grid_for(total, kThreads), kThreads, 0, st>>>(
        static_cast<const uint32_t*>(src), static_cast<uint32_t*>(dst), outer, d_src, src_off, d_dst, dst_off, count, inner);
  } else {
    copy_dim_block<uint16_t><<<grid_for(total, kThreads), kThreads, 0, st>>>(
        static_cast<const uint16_t*>(src), static_cast<uint16_t*>(dst), outer, d_src, src_off, d_dst, dst_off, count, inner);
  }
  return launch_status();
}

void fill_win_params(const gl_ap* in, const gl_windows* w, const gl_ap& A, WinParams* p) {
  std::memset(p, 0, sizeof(*p));
  const int na = in->access_ndim;
  p->n = w->n;
  int64_t s = 1;
  p->wcells = 1;
  for (int i = w->n - 1; i >= 0; --i) {
    p->in_size[i] = in->shape[na + i];
    p->in_stride[i] = s;
    s *= in->shape[na + i];
    p->out_ext[i] = A.shape[na + i];
    p->w[i] = w->wshape[i];
    p->s[i] = w->stride[i];
    p->pad_lo[i] = w->pad_lo[i];
    p->wcells *= w->wshape[i];
  }
  p->item = s;
  p->total = numel(A);
}

int device_smem_optin() {
  static int cached = 0;   // the same value on every GPU of a node
  if (cached) return cached;
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return 0;
  cached = v;
  return v;
}

constexpr int kIm2colMaxSmem = 160 * 1024;

// Raises the kernel's dynamic shared-memory limit once (per process) instead of on every call.
template <typename K>
bool allow_big_smem(K kern, bool* done) {
  if (*done) return true;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kIm2colMaxSmem) != cudaSuccess) return false;
  *done = true;
  return true;
}

template <typename T>
int run_windows(const gl_ap* in, const gl_windows* w, const gl_ap& A, gl_ap* out, cudaStream_t st) {
  constexpr int VEC = 16 / sizeof(T);
  const T fill = Fill<T>::value(w->pad_kind);
  const T* src = static_cast<const T*>(in->data);
  T* dst = static_cast<T*>(out->data);
  const int na = in->access_ndim;
  const int64_t* b = in->shape + na;
  // convolution-style fast path: window spans the whole first compute dim
  if (w->n == 3 && w->wshape[0] == b[0] && w->pad_lo[0] == 0 && w->pad_hi[0] == 0) {
    Im2colParams p;
    p.N = prod(in->shape, 0, na);
    p.C = b[0]; p.H = b[1]; p.W = b[2];
    p.Kh = w->wshape[1]; p.Kw = w->wshape[2];
    p.Sh = w->stride[1]; p.Sw = w->stride[2];
    p.ph_lo = w->pad_lo[1]; p.pw_lo = w->pad_lo[2];
    p.Ho = A.shape[na + 1]; p.Wo = A.shape[na + 2];
    p.K = p.C * p.Kh * p.Kw;
    // rows that are whole 16-byte pieces are staged 16-byte aligned behind a margin of one piece
    // (4-byte elements only: a pitch of whole pieces puts the 2-byte gather on few banks)
    const bool aligned = sizeof(T) == 4 && p.W % VEC == 0 && w->pad_lo[2] <= VEC;
    const int64_t wp = p.W + (aligned ? VEC : w->pad_lo[2]) + w->pad_hi[2];
    // Two blocks per (n, h'), half the channels each, when the halves of an output row are whole 128-byte
    // lines: the same work in more, shorter blocks (a shorter last wave, more warps per SM in flight).
    p.cparts = (p.C % 2 == 0 && (p.K / 2 * sizeof(T)) % 128 == 0 && p.N * p.Ho < (1ll << 30)) ? 2 : 1;
    const int64_t Kb = p.K / p.cparts, rows_b = p.C / p.cparts * p.Kh;
    const bool vec = Kb % VEC == 0;
    const int pitch = wp < (1 << 20) && p.K < (1 << 24)
                          ? best_im2col_pitch(static_cast<int>(wp), static_cast<int>(p.Kw), static_cast<int>(Kb),
                                              vec ? VEC : 1, static_cast<int>(sizeof(T)), aligned ? VEC : 1)
                          : static_cast<int>((wp + VEC - 1) / VEC * VEC);
    const int64_t smem = (((Kb + rows_b) * 4 + 15) / 16) * 16 + rows_b * pitch * (int64_t)sizeof(T);
    const int64_t blocks = p.N * p.Ho * p.cparts;
    if (smem <= kIm2colMaxSmem && smem <= device_smem_optin() && blocks <= 0x7FFFFFFF && p.Wo * p.K < (1ll << 30) &&
        p.C * p.H * p.W < (1ll << 31)) {
      p.Wp = static_cast<int>(wp);
      p.pitch = pitch;
      p.aligned = aligned ? 1 : 0;
      p.Cb = static_cast<int>(p.C / p.cparts);
      p.Kb = static_cast<int>(Kb);
      p.by_Ho = make_fastdiv(p.Ho); p.by_Kh = make_fastdiv(p.Kh); p.by_Kw = make_fastdiv(p.Kw);
      p.by_border = make_fastdiv(std::max<int64_t>(1, wp - p.W - (aligned ? VEC : w->pad_lo[2]) + w->pad_lo[2]));
      p.by_wv = make_fastdiv(std::max<int64_t>(1, p.W / VEC));
      p.lg = 0;
      while ((1 << p.lg) < p.W / VEC && p.lg < 5) ++p.lg;
      p.dc = static_cast<int>((kThreads >> p.lg) / p.Kh);
      p.dkh = static_cast<int>((kThreads >> p.lg) - p.dc * p.Kh);
      p.groups = p.segs = 1;
      p.rsplit = p.gsplit = 0;
      p.by_segs = make_fastdiv(1);
      p.slide = 0;
      if (vec && sizeof(T) == 4 && p.Sw == 1 && p.Kw >= 3 && p.Wo >= 2) {
        // item length that minimises (rounds over the block's quarter warps) x (loads per item); odd
        // lengths only (see the kernel)
        const int64_t groups = (Kb / 4 + 7) / 8, nq = kThreads / 8;
        int64_t best_cost = INT64_MAX;
        for (int64_t L = p.Wo >= 3 ? 3 : 1; L <= p.Wo; L += 2) {
          const int64_t items = groups * ((p.Wo + L - 1) / L);
          const int64_t cost = ((items + nq - 1) / nq) * (2 * L + 2);
          if (cost < best_cost) { best_cost = cost; p.slide = static_cast<int>(L); }
        }
        p.groups = static_cast<int>(groups);
        p.segs = static_cast<int>((p.Wo + p.slide - 1) / p.slide);
        p.by_segs = make_fastdiv(p.segs);
        if (aligned && p.Cb >= 2) {
          p.rsplit = static_cast<int>(p.Cb / 2 * p.Kh);
          p.gsplit = static_cast<int>(p.rsplit * p.Kw / 32);   // a group is 32 columns; column k reads row k / Kw
        }
      }
      auto kern = vec ? im2col_rows<T, VEC> : im2col_rows<T, 1>;
      static bool attr_done[64][2] = {{false}};   // per device and kernel variant
      int dev = 0;
      if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return GL_ERR_CUDA;
      if (!allow_big_smem(kern, &attr_done[dev][vec ? 1 : 0])) return GL_ERR_CUDA;
      return launch_pdl(kern, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), static_cast<size_t>(smem), st, 1, src,
                        dst, p, fill) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
    }
  }
  WinParams p;
  fill_win_params(in, w, A, &p);
  windows_generic<T><<<grid_for(p.total, kThreads), kThreads, 0, st>>>(src, dst, p, fill);
  return launch_status();
}

}  // namespace

extern "C" {

int gl_access_transpose(const gl_ap* in, const int32_t* perm, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out || !perm) return GL_ERR_NULL;
  gl_ap want = *in;
  rc = gl_shape_transpose(in, perm, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return in->dtype == GL_F32 ? run_transpose<uint32_t>(in, perm, out, st) : run_transpose<uint16_t>(in, perm, out, st);
}

int gl_access_pad(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, int32_t pad_kind, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (pad_kind != GL_PAD_ZERO && pad_kind != GL_PAD_NEG_INF) return GL_ERR_SHAPE;
  gl_ap want = *in;
  rc = gl_shape_pad(in, dim, lo, hi, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t outer = prod(in->shape, 0, dim), inner = prod(in->shape, dim + 1, in->ndim);
  const int64_t d_in = in->shape[dim], d_out = d_in + lo + hi;
  const size_t es = dtype_size(in->dtype);
  const int vec = static_cast<int>(16 / es);
  if (inner % vec == 0) {
    uint4 fill;
    const uint32_t f32 = Fill<uint32_t>::value(pad_kind);
    const uint32_t f16 = Fill<uint16_t>::value(pad_kind) * 0x10001u;
    fill.x = fill.y = fill.z = fill.w = (in->dtype == GL_F32 ? f32 : f16);
    const int64_t total = outer * d_out * (inner / vec);
    pad_kernel<uint4><<<grid_for(total, kThreads), kThreads, 0, st>>>(
        static_cast<const uint4*>(in->data), static_cast<uint4*>(out->data), outer, d_in, lo, d_out, inner / vec, fill);
  } else if (inner == 1 && d_out < (1ll << 30)) {
    const unsigned blocks = static_cast<unsigned>(std::min<int64_t>((outer + 7) / 8, 148 * 32));
    if (in->dtype == GL_F32 && d_out <= 512 && outer * d_out < (1ll << 31)) {
      // multiply-high division by d_out for n < 2^31: p = ceil(log2 d), m = ceil(2^(31+p) / d), n / d = umulhi(n, m) >> (p - 1)
      uint32_t pw2 = 0;
      while ((1ull << pw2) < static_cast<uint64_t>(d_out)) ++pw2;
      const uint32_t mul = pw2 ? static_cast<uint32_t>(((1ull << (31 + pw2)) + d_out - 1) / d_out) : 0u;
      const int64_t total = outer * d_out;
      const unsigned fblocks = static_cast<unsigned>(std::min<int64_t>((total / 4 + kThreads - 1) / kThreads + 1, 148 * 32));
      return launch_pdl(pad_rows_flat, dim3(fblocks), dim3(kThreads), 0, st, 1, static_cast<const uint32_t*>(in->data),
                        static_cast<uint32_t*>(out->data), total, (int)d_in, (int)lo, (int)d_out, mul,
                        pw2 ? pw2 - 1 : 0u, Fill<uint32_t>::value(pad_kind)) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
    }
    if (in->dtype == GL_F32)
      return launch_pdl(pad_rows<uint32_t>, dim3(blocks), dim3(kThreads), 0, st, 1, static_cast<const uint32_t*>(in->data),
                        static_cast<uint32_t*>(out->data), outer, (int)d_in, (int)lo, (int)d_out,
                        Fill<uint32_t>::value(pad_kind)) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
    else
      return launch_pdl(pad_rows<uint16_t>, dim3(blocks), dim3(kThreads), 0, st, 1, static_cast<const uint16_t*>(in->data),
                        static_cast<uint16_t*>(out->data), outer, (int)d_in, (int)lo, (int)d_out,
                        Fill<uint16_t>::value(pad_kind)) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  } else if (in->dtype == GL_F32) {
    pad_kernel<uint32_t><<<grid_for(outer * d_out * inner, kThreads), kThreads, 0, st>>>(
        static_cast<const uint32_t*>(in->data), static_cast<uint32_t*>(out->data), outer, d_in, lo, d_out, inner,
        Fill<uint32_t>::value(pad_kind));
  } else {
    pad_kernel<uint16_t><<<grid_for(outer * d_out * inner, kThreads), kThreads, 0, st>>>(
        static_cast<const uint16_t*>(in->data), static_cast<uint16_t*>(out->data), outer, d_in, lo, d_out, inner,
        Fill<uint16_t>::value(pad_kind));
  }
  return launch_status();
}

int gl_access_windows(const gl_ap* in, const gl_windows* w, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out || !w) return GL_ERR_NULL;
  gl_ap want = *in;
  rc = gl_shape_windows(in, w, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return in->dtype == GL_F32 ? run_windows<uint32_t>(in, w, want, out, st) : run_windows<uint16_t>(in, w, want, out, st);
}

int gl_compute_reduce_max(const gl_ap* in, const gl_windows* w, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (in->dtype != GL_F32 && in->dtype != GL_BF16) return GL_ERR_DTYPE;
  gl_ap want = *in;
  rc = gl_shape_reduce_max(in, w, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float* src = static_cast<const float*>(in->data);
  float* dst = static_cast<float*>(out->data);
  const bool bf16 = in->dtype == GL_BF16;
  if (w) {
    // channels-last items (H,W,C) with window (Kh,Kw,1), stride (Sh,Sw,1), no pad on C: 16-byte channel pieces
    const int nc = in->access_ndim;
    const int64_t per_piece = bf16 ? 8 : 4;
    if (w->n == 3 && w->wshape[2] == 1 && w->stride[2] == 1 && w->pad_lo[2] == 0 && w->pad_hi[2] == 0 &&
        in->shape[nc + 2] % per_piece == 0 && in->shape[nc] < (1 << 20) && in->shape[nc + 1] < (1 << 20)) {
      gl_ap A = *in;
      gl_shape_windows(in, w, &A);
      PoolHwc t;
      t.H = (int)in->shape[nc]; t.W = (int)in->shape[nc + 1];
      t.Kh = (int)w->wshape[0]; t.Kw = (int)w->wshape[1];
      t.Sh = (int)w->stride[0]; t.Sw = (int)w->stride[1];
      t.ph = (int)w->pad_lo[0]; t.pw = (int)w->pad_lo[1];
      t.Ho = (int)A.shape[nc]; t.Wo = (int)A.shape[nc + 1];
      t.cv = (int)(in->shape[nc + 2] / per_piece);
      const int64_t pieces = prod(in->shape, 0, nc) * t.Ho * t.Wo * t.cv;
      // few outputs with large windows: up to 32 lanes per output piece, while that leaves every lane four cells
      // and the machine is not yet full
      t.split_log2 = 0;
      while (t.split_log2 < 5 && (t.Kh * t.Kw >> (t.split_log2 + 1)) >= 4 && (pieces << t.split_log2) < 148 * 2048 * 2) ++t.split_log2;
      t.total = pieces << t.split_log2;
      if (t.total < (1ll << 31)) {
        t.by_Kw = make_fastdiv(t.Kw);
        t.by_cv = make_fastdiv(t.cv);
        t.by_Wo = make_fastdiv(t.Wo);
        t.by_Ho = make_fastdiv(t.Ho);
        const float fill = w->pad_kind == GL_PAD_NEG_INF ? -INFINITY : 0.0f;
        if (t.split_log2 == 0 && t.Kh == 3 && t.Kw == 3 && (t.total + kThreads - 1) / kThreads <= 0x7FFFFFFF) {
          const dim3 fgrid(static_cast<unsigned>((t.total + kThreads - 1) / kThreads));
          const cudaError_t ferr =
              bf16 ? launch_pdl(window_max_hwc_fixed<true, 3, 3>, fgrid, dim3(kThreads), 0, st, 1,
                                static_cast<const uint4*>(in->data), static_cast<uint4*>(out->data), t, fill)
                   : launch_pdl(window_max_hwc_fixed<false, 3, 3>, fgrid, dim3(kThreads), 0, st, 1,
                                static_cast<const uint4*>(in->data), static_cast<uint4*>(out->data), t, fill);
          return ferr == cudaSuccess ? GL_OK : GL_ERR_CUDA;
        }
        const dim3 grid(grid_for(t.total, kThreads));
        const cudaError_t err =
            bf16 ? launch_pdl(window_max_hwc<true>, grid, dim3(kThreads), 0, st, 1, static_cast<const uint4*>(in->data),
                              static_cast<uint4*>(out->data), t, fill)
                 : launch_pdl(window_max_hwc<false>, grid, dim3(kThreads), 0, st, 1, static_cast<const uint4*>(in->data),
                              static_cast<uint4*>(out->data), t, fill);
        return err == cudaSuccess ? GL_OK : GL_ERR_CUDA;
      }
    }
  }
  if (bf16) {
    // 2-byte planes ((..),(H,W)): the tiled kernel, else the plain one; other bf16 forms have no kernel
    const int nb = in->access_ndim;
    if (!w || w->n != 2 || in->shape[nb] >= (1 << 30) || in->shape[nb + 1] >= (1 << 30)) return GL_ERR_UNSUPPORTED;
    gl_ap A = *in;
    gl_shape_windows(in, w, &A);
    const float fill = w->pad_kind == GL_PAD_NEG_INF ? -INFINITY : 0.0f;
    const int64_t nwin = numel(want);
    if (w->wshape[0] == 3 && w->wshape[1] == 3 && w->stride[0] == 2 && w->stride[1] == 2 && w->pad_lo[0] == 1 &&
        w->pad_lo[1] == 1 && in->shape[nb + 1] % 8 == 0 && in->shape[nb] < (1 << 20) && in->shape[nb + 1] < (1 << 20) &&
        A.shape[nb + 1] * 2 == in->shape[nb + 1]) {
      constexpr int kRows = 2;
      Pool3s2H t;
      t.H = (int)in->shape[nb]; t.W = (int)in->shape[nb + 1];
      t.Ho = (int)A.shape[nb]; t.Wo = (int)A.shape[nb + 1];
      t.strips = (t.Ho + kRows - 1) / kRows;
      t.w8 = t.W / 8;
      t.items = prod(in->shape, 0, nb) * t.strips * t.w8;
      if (t.items < (1ll << 31)) {
        t.by_w8 = make_fastdiv(t.w8);
        t.by_strips = make_fastdiv(t.strips);
        return launch_pdl(window_max_3x3s2_bf16<kRows>, dim3(static_cast<unsigned>((t.items + 255) / 256)), dim3(256), 0, st, 1,
                          static_cast<const uint16_t*>(in->data), static_cast<uint16_t*>(out->data), t, fill) == cudaSuccess
                   ? GL_OK : GL_ERR_CUDA;
      }
    }
    if (w->wshape[1] == 8 && w->stride[1] == 8 && w->pad_lo[1] == 0 && in->shape[nb + 1] % 8 == 0 &&
        A.shape[nb + 1] * 8 <= in->shape[nb + 1] && w->wshape[0] <= 64 && w->stride[0] < 1024 && w->pad_lo[0] < 1024 &&
        in->shape[nb] < (1 << 20) && in->shape[nb + 1] < (1 << 20) && nwin < (1ll << 31)) {
      PoolRow8 t;
      t.H = (int)in->shape[nb]; t.W = (int)in->shape[nb + 1];
      t.Kh = (int)w->wshape[0]; t.Sh = (int)w->stride[0]; t.ph = (int)w->pad_lo[0];
      t.Ho = (int)A.shape[nb]; t.Wo = (int)A.shape[nb + 1];
      t.total = nwin;
      t.by_Wo = make_fastdiv(t.Wo);
      t.by_Ho = make_fastdiv(t.Ho);
      return launch_pdl(window_max_rows8_bf16, dim3(static_cast<unsigned>((nwin + kThreads - 1) / kThreads)), dim3(kThreads), 0, st,
                        1, static_cast<const uint16_t*>(in->data), static_cast<uint16_t*>(out->data), t, fill) == cudaSuccess
                 ? GL_OK : GL_ERR_CUDA;
    }
    if (in->shape[nb] < (1 << 20) && in->shape[nb + 1] < (1 << 20) && w->wshape[0] < 1024 && w->wshape[1] < 1024 &&
        w->stride[0] < 1024 && w->stride[1] < 1024) {
      PoolTile t;
      if (plan_pool_tile(in, w, A, nb, 8, &t)) {
        const int rows = (t.TH - 1) * t.Sh + t.Kh;
        window_max_2d_tiled<uint16_t><<<static_cast<unsigned>(prod(in->shape, 0, nb) * t.tiles), kThreads,
                                        static_cast<size_t>(rows) * t.Wp * 4, st>>>(
            static_cast<const uint16_t*>(in->data), static_cast<uint16_t*>(out->data), t, fill);
        return launch_status();
      }
    }
    return launch_pdl(window_max_2d_bf16, dim3(grid_for(nwin, kThreads)), dim3(kThreads), 0, st, 1,
                      static_cast<const uint16_t*>(in->data), static_cast<uint16_t*>(out->data), prod(in->shape, 0, nb),
                      (int)in->shape[nb], (int)in->shape[nb + 1], (int)w->wshape[0], (int)w->wshape[1], (int)w->stride[0],
                      (int)w->stride[1], (int)w->pad_lo[0], (int)w->pad_lo[1], (int)A.shape[nb], (int)A.shape[nb + 1],
                      fill) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
  }
  if (!w) {
    const int64_t items = prod(in->shape, 0, in->access_ndim), item = prod(in->shape, in->access_ndim, in->ndim);
    item_max<<<grid_for(items, kThreads / 32), kThreads, 0, st>>>(src, dst, items, item);
    return launch_status();
  }
  gl_ap A = *in;
  gl_shape_windows(in, w, &A);
  const float fill = w->pad_kind == GL_PAD_NEG_INF ? -INFINITY : 0.0f;
  const int64_t nwin = numel(want);
  const int na = in->access_ndim;
  if (w->n == 2 && w->wshape[0] == 3 && w->wshape[1] == 3 && w->stride[0] == 2 && w->stride[1] == 2 &&
      w->pad_lo[0] == 1 && w->pad_lo[1] == 1 && in->shape[na + 1] % 4 == 0 && in->shape[na] < (1 << 20) &&
      in->shape[na + 1] < (1 << 20) && A.shape[na + 1] % 2 == 0) {
    Pool3s2 t;
    t.H = (int)in->shape[na]; t.W = (int)in->shape[na + 1];
    t.Ho = (int)A.shape[na]; t.Wo = (int)A.shape[na + 1];
    constexpr int kRows = 2;   // short strips: more threads in flight beat the shared odd rows (measured)
    t.R = kRows;
    t.strips = (t.Ho + t.R - 1) / t.R;
    t.w4 = t.W / 4;
    t.units = prod(in->shape, 0, na) * t.strips;
    t.by_strips = make_fastdiv(t.strips);
    const int64_t items = t.units * t.w4;
    if (t.w4 % 32 != 0 && items < (1ll << 31)) {
      return launch_pdl(window_max_3x3s2_flat<kRows>, dim3(static_cast<unsigned>((items + 255) / 256)), dim3(256), 0, st, 1, src, dst,
                        t, items, make_fastdiv(t.w4), fill) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
    }
    const int64_t blocks = (t.units + 7) / 8;
    if (blocks <= 0x7FFFFFFF) {
      return launch_pdl(window_max_3x3s2<kRows>, dim3(static_cast<unsigned>(blocks)), dim3(32, 8), 0, st, 1, src, dst, t,
                        fill) == cudaSuccess ? GL_OK : GL_ERR_CUDA;
    }
  }
  if (w->n == 2 && in->shape[na] < (1 << 20) && in->shape[na + 1] < (1 << 20) && w->wshape[0] < 1024 &&
      w->wshape[1] < 1024 && w->stride[0] < 1024 && w->stride[1] < 1024) {
    PoolTile t;
    if (plan_pool_tile(in, w, A, na, 4, &t)) {
      const int rows = (t.TH - 1) * t.Sh + t.Kh;
      window_max_2d_tiled<float><<<static_cast<unsigned>(prod(in->shape, 0, na) * t.tiles), kThreads,
                                   static_cast<size_t>(rows) * t.Wp * 4, st>>>(src, dst, t, fill);
      return launch_status();
    }
  }
  if (w->n == 2 && in->shape[na] < (1 << 30) && in->shape[na + 1] < (1 << 30)) {
    window_max_2d<<<grid_for(nwin, kThreads), kThreads, 0, st>>>(
        src, dst, prod(in->shape, 0, na), (int)in->shape[na], (int)in->shape[na + 1], (int)w->wshape[0],
        (int)w->wshape[1], (int)w->stride[0], (int)w->stride[1], (int)w->pad_lo[0], (int)w->pad_lo[1],
        (int)A.shape[na], (int)A.shape[na + 1], fill);
    return launch_status();
  }
  WinParams p;
  fill_win_params(in, w, A, &p);
  window_max_generic<<<grid_for(nwin, kThreads), kThreads, 0, st>>>(src, dst, p, nwin, fill);
  return launch_status();
}

int gl_access_slice(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  gl_ap want = *in;
  rc = gl_shape_slice(in, dim, lo, hi, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  return run_copy_dim(in->data, out->data, in->dtype, prod(in->shape, 0, dim), in->shape[dim], lo, hi - lo, 0, hi - lo,
                      prod(in->shape, dim + 1, in->ndim), static_cast<cudaStream_t>(stream));
}

int gl_access_concat(const gl_ap* a, const gl_ap* b, int32_t dim, gl_ap* out, void* stream) {
  int rc = check_data(a);
  if (rc) return rc;
  rc = check_data(b);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  gl_ap want = *a;
  rc = gl_shape_concat(a, b, dim, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t outer = prod(a->shape, 0, dim), inner = prod(a->shape, dim + 1, a->ndim);
  const int64_t da = a->shape[dim], db = b->shape[dim];
  rc = run_copy_dim(a->data, out->data, a->dtype, outer, da, 0, da + db, 0, da, inner, st);
  if (rc) return rc;
  return run_copy_dim(b->data, out->data, a->dtype, outer, db, 0, da + db, da, db, inner, st);
}

int gl_access_pair(const gl_ap* a, const gl_ap* b, gl_ap* out, void* stream) {
  int rc = check_data(a);
  if (rc) return rc;
  rc = check_data(b);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  gl_ap want = *a;
  rc = gl_shape_pair(a, b, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t outer = prod(a->shape, 0, a->access_ndim), inner = prod(a->shape, a->access_ndim, a->ndim);
  rc = run_copy_dim(a->data, out->data, a->dtype, outer, 1, 0, 2, 0, 1, inner, st);
  if (rc) return rc;
  return run_copy_dim(b->data, out->data, a->dtype, outer, 1, 0, 2, 1, 1, inner, st);
}

int gl_compute_reduce_sum(const gl_ap* in, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (in->dtype != GL_F32) return GL_ERR_DTYPE;
  gl_ap want = *in;
  rc = gl_shape_reduce_sum(in, &want);
  if (rc) return rc;
  rc = check_same_meta(want, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  const int64_t items = prod(in->shape, 0, in->access_ndim), item = prod(in->shape, in->access_ndim, in->ndim);
  item_sum<<<grid_for(items, kThreads / 32), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const float*>(in->data), static_cast<float*>(out->data), items, item);
  return launch_status();
}

int gl_compute_relu(const gl_ap* in, gl_ap* out, void* stream) {
  int rc = check_data(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (in->dtype != GL_F32) return GL_ERR_DTYPE;
  rc = check_same_meta(*in, out);
  if (rc) return rc;
  rc = check_data(out);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t n = numel(*in), n4 = n / 4;
  const float* src = static_cast<const float*>(in->data);
  float* dst = static_cast<float*>(out->data);
  if (n4) {
    int64_t blocks = (n4 + kThreads - 1) / kThreads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (launch_pdl(relu_vec, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, st, 1,
                   reinterpret_cast<const float4*>(src), reinterpret_cast<float4*>(dst), n4) != cudaSuccess)
      return GL_ERR_CUDA;
  }
  if (n % 4) relu_tail<<<1, 4, 0, st>>>(src, dst, n4 * 4, n);
  return launch_status();
}

}  // extern "C"
