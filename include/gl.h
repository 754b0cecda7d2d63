/*
 * gl.h - C ABI of the access-pattern evaluator for B200 (sm_100a).
 *
 * The calls follow the operators of "Pure Tensor Program Rewriting via Access
 * Patterns" (Glenside): the access-pattern transformers of Section 4.2 (first
 * table of Section 4) and the operators applied by `compute` (Section 4.3,
 * operator table).  An access pattern is a dense row-major tensor whose
 * dimensions are split into access dimensions S_A (iterated over) and compute
 * dimensions S_C (computed on); its tensor shape is S_A ++ S_C (Section 4.1).
 *
 * Conventions for every call
 *   - Return value: GL_OK or a GL_ERR_* code; gl_strerror() names it.
 *   - All arguments are validated, and every descriptor a call needs is prepared,
 *     before anything is enqueued: a call that returns any error other than a
 *     failed kernel launch has launched nothing and written nothing.  (A launch
 *     that the runtime itself refuses, GL_ERR_CUDA, may follow an earlier launch
 *     of the same call, which has then written the workspace but not `out`.)
 *   - gl_shape_* calls are host-only: they read shapes, never `data`.
 *   - Device calls enqueue kernels on `stream` (a cudaStream_t passed as
 *     void*, NULL = the default stream).  They never synchronise and never
 *     allocate.  `data` pointers are DEVICE pointers owned by the caller, who
 *     also owns outputs and workspaces.  `out->shape`, `out->ndim`,
 *     `out->access_ndim` and `out->dtype` must already equal what the matching
 *     gl_shape_* call returns, otherwise GL_ERR_SHAPE / GL_ERR_DTYPE.
 *   - Inputs are read-only and must not overlap outputs (gl_compute_relu may
 *     run in place).  Data pointers must be 16-byte aligned (GL_ERR_ALIGN).
 *   - There is no CPU fallback: a combination the kernels do not cover
 *     returns GL_ERR_UNSUPPORTED.
 *   - Calls are re-entrant from several host threads.
 */
#ifndef GL_H_
#define GL_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define GL_API __attribute__((visibility("default")))
#else
#define GL_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
  GL_OK = 0,
  GL_ERR_NULL = 1,        /* a required pointer is NULL                              */
  GL_ERR_DTYPE = 2,       /* dtype not accepted by this call                         */
  GL_ERR_NDIM = 3,        /* ndim / access_ndim out of range                         */
  GL_ERR_SHAPE = 4,       /* shapes disagree (with each other or with gl_shape_*)    */
  GL_ERR_PERM = 5,        /* not a permutation of 0..ndim-1                          */
  GL_ERR_ALIGN = 6,       /* a data pointer is not 16-byte aligned                   */
  GL_ERR_UNSUPPORTED = 7, /* valid program, but no kernel covers it                  */
  GL_ERR_WORKSPACE = 8,   /* workspace missing or smaller than the _workspace() size */
  GL_ERR_CUDA = 9,        /* the CUDA runtime or driver reported an error            */
  GL_ERR_TIMEOUT = 10     /* a bounded wait inside a kernel gave up                  */
};

enum { GL_BF16 = 1, GL_F32 = 2 };
enum { GL_PAD_ZERO = 0, GL_PAD_NEG_INF = 1 };

#define GL_MAX_DIMS 8

/* Access pattern (Section 4.1): tensor of shape S_A ++ S_C, dense, row-major. */
typedef struct {
  void* data;          /* device pointer (ignored by gl_shape_*)                 */
  int32_t dtype;       /* GL_BF16 or GL_F32                                       */
  int32_t ndim;        /* |S_A| + |S_C|, 0..GL_MAX_DIMS                           */
  int32_t access_ndim; /* |S_A|: `(access T access_ndim)`                         */
  int32_t reserved_;
  int64_t shape[GL_MAX_DIMS];
} gl_ap;

/* Arguments of `windows` (transformer table): one window extent and one
 * stride per COMPUTE dimension of the input.  pad_lo / pad_hi describe a
 * `pad` of that compute dimension applied first (pad is not in the paper;
 * it is the constant border that ML convolutions and pools use): the padded
 * tensor is never written, out-of-range cells read as the fill value. */
typedef struct {
  int32_t n;        /* number of compute dims of the input = ndim - access_ndim */
  int32_t pad_kind; /* GL_PAD_ZERO or GL_PAD_NEG_INF                             */
  int64_t wshape[GL_MAX_DIMS];
  int64_t stride[GL_MAX_DIMS];
  int64_t pad_lo[GL_MAX_DIMS];
  int64_t pad_hi[GL_MAX_DIMS];
} gl_windows;

/* Flags of gl_cartesian_dot */
#define GL_EPILOGUE_RELU 0x2u       /* apply compute relu to every result before it is stored  */
#define GL_OUT_NCHW 0x4u             /* conv2d only: store transpose(squeeze(...)) of Fig. 2a, i.e.
                                        ((N, O, H', W'),()); see gl_shape_cartesian_dot_nchw      */
#define GL_OUT_BF16 0x8u             /* store the results rounded to bf16 (nearest even) instead of fp32: `out`
                                      * must then be GL_BF16.  Sums are still carried in fp32; the rounding is
                                      * the last step, after relu.  Lets the next layer read its operand as is
                                      * and halves the bytes written. */
#define GL_DOT_GENERAL_KERNEL 0x100u /* skip the tensor-core path: run the general kernel, which
                                        takes any shape and sums each window in index order      */

/* ----------------------------------------------------------------------- */
/* Host-only shape inference.  Each fills out->ndim, access_ndim, shape and  */
/* dtype (copied from the input, GL_F32 for dot products) and leaves         */
/* out->data untouched.                                                      */
/* ----------------------------------------------------------------------- */

/* `access` (transformer table, row 1): move the split to position i. */
GL_API int gl_shape_access(const gl_ap* in, int32_t i, gl_ap* out);

/* `windows` (transformer table): ((a..),(b_0..b_n)) -> ((a.., b'_0..b'_n),(w_0..w_n)),
 * b'_i = ceil((b_i + pad_lo_i + pad_hi_i - (w_i - 1)) / s_i).  A window larger than
 * its padded dimension, or a pad not smaller than the window, is GL_ERR_SHAPE. */
GL_API int gl_shape_windows(const gl_ap* in, const gl_windows* w, gl_ap* out);

/* `flatten` (transformer table): ((prod a),(prod b)); a side without dims stays empty. */
GL_API int gl_shape_flatten(const gl_ap* in, gl_ap* out);

/* `transpose` (transformer table, Section 4.2): output dim j = input dim perm[j];
 * perm covers all ndim dims; the split position is kept. */
GL_API int gl_shape_transpose(const gl_ap* in, const int32_t* perm, gl_ap* out);

/* `pad` (not in the paper): dimension `dim` grows by lo + hi. */
GL_API int gl_shape_pad(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, gl_ap* out);

/* `slice` (transformer table): dimension `dim` keeps [lo, hi). */
GL_API int gl_shape_slice(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, gl_ap* out);

/* `concat` (used by the blocking rewrites of Section 5.4, Fig. 7): join a and b along `dim`; all
 * other extents, the split position and the dtype must agree. */
GL_API int gl_shape_concat(const gl_ap* a, const gl_ap* b, int32_t dim, gl_ap* out);

/* `pair` (transformer table): two patterns of one shape -> ((a..),(2, c..)). */
GL_API int gl_shape_pair(const gl_ap* a, const gl_ap* b, gl_ap* out);

/* `squeeze` (transformer table): drop dimension `dim`, which must have extent 1.  Metadata only:
 * the data of the result is the data of the input. */
GL_API int gl_shape_squeeze(const gl_ap* in, int32_t dim, gl_ap* out);

/* `reshape` (transformer table): new shape `shape[0..ndim)` split at `access_ndim`; the element
 * counts of the access side and of the compute side must both be kept.  Metadata only. */
GL_API int gl_shape_reshape(const gl_ap* in, const int64_t* shape, int32_t ndim, int32_t access_ndim, gl_ap* out);

/* compute reduceSum (operator table): ((access dims),()). */
GL_API int gl_shape_reduce_sum(const gl_ap* in, gl_ap* out);

/* compute dotProd (cartProd (windows? a0) a1)  (Section 4.2 cartProd, Section 4.3
 * dotProd, Fig. 2a/2b): with A = windows(a0) (or a0 itself when w is NULL) of shape
 * ((m..),(k..)) and a1 of shape ((o..),(k..)), the result is ((m.., o..),()), GL_F32. */
GL_API int gl_shape_cartesian_dot(const gl_ap* a0, const gl_windows* w_or_null, const gl_ap* a1, gl_ap* out);

/* The whole conv2d of Fig. 2a: transpose (squeeze (compute dotProd (cartProd (windows a0) a1)) 1)
 * (0 3 1 2).  a0 must be ((n..),(C,H,W)) with window (C,Kh,Kw), or ((n..),(H,W,C)) with window
 * (Kh,Kw,C); the result is ((n.., o.., H', W'),()), GL_F32: the window-position dims move behind
 * the filter dims and the size-1 channel position is squeezed away.  This is the shape
 * gl_cartesian_dot expects for `out` when GL_OUT_NCHW is set. */
GL_API int gl_shape_cartesian_dot_nchw(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, gl_ap* out);

/* compute reduceMax (windows? in) (operator table; Fig. 2c): ((access dims of A),()). */
GL_API int gl_shape_reduce_max(const gl_ap* in, const gl_windows* w_or_null, gl_ap* out);

/* ----------------------------------------------------------------------- */
/* Device operations                                                         */
/* ----------------------------------------------------------------------- */

/* Materialised `windows` (transformer table; Section 5.3 calls the result, once
 * flattened, the im2col matrix): out[a.., p.., q..] = in[a.., p_i*s_i + q_i - pad_lo_i],
 * the fill value where that index is outside the input.  GL_F32 or GL_BF16. */
GL_API int gl_access_windows(const gl_ap* in, const gl_windows* w, gl_ap* out, void* stream);

/* `flatten` is metadata on dense data: fills out's shape and sets out->data = in->data. */
GL_API int gl_access_flatten(const gl_ap* in, gl_ap* out);

/* `transpose` with data movement: out[i_0..] = in[j_0..] with j_{perm[d]} = i_d.
 * GL_F32 or GL_BF16, any rank up to GL_MAX_DIMS. */
GL_API int gl_access_transpose(const gl_ap* in, const int32_t* perm, gl_ap* out, void* stream);

/* Materialised `pad` of one dimension with 0 or -inf (not in the paper). */
GL_API int gl_access_pad(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, int32_t pad_kind,
                  gl_ap* out, void* stream);

/* `slice`, `concat`, `pair` with data movement (transformer table; Fig. 7).  GL_F32 or GL_BF16. */
GL_API int gl_access_slice(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, gl_ap* out, void* stream);
GL_API int gl_access_concat(const gl_ap* a, const gl_ap* b, int32_t dim, gl_ap* out, void* stream);
GL_API int gl_access_pair(const gl_ap* a, const gl_ap* b, gl_ap* out, void* stream);

/* compute reduceSum (operator table): the sum of every item, GL_F32, added in a fixed order (a
 * strided partial sum per lane of one warp, then a butterfly), so results repeat bit for bit. */
GL_API int gl_compute_reduce_sum(const gl_ap* in, gl_ap* out, void* stream);

/* out = compute dotProd (cartProd (windows? a0) a1), optionally followed by compute
 * relu (Fig. 2a for conv2d with w given, Fig. 2b / Fig. 6 for matrix products with
 * w NULL).  a0 and a1 are GL_BF16, products and sums are carried in fp32, out is
 * GL_F32 (GL_BF16 with GL_OUT_BF16) with the access dims of A followed by those of a1,
 * i.e. row-major [M, O].
 * Two item layouts take the tensor-core path:
 *   - w NULL, a0 ((M),(K)), a1 ((O),(K)) with K a multiple of 8;
 *   - a0 ((N),(C,H,W)) with window (C,Kh,Kw), stride (1,Sh,Sw), or a0 ((N),(H,W,C))
 *     with window (Kh,Kw,C), stride (Sh,Sw,1); a1 ((O),(same item shape as the window)).
 * Everything else runs on a slower general kernel.  The sum over the window is
 * taken in an unspecified order.  `workspace` must hold at least
 * gl_cartesian_dot_workspace() bytes (it may be NULL when that is 0) and must be
 * 1024-byte aligned; its contents are scratch.  Few-channel convolutions (at most
 * 8 / Sw channels, the RGB stem), channels-last items with a channel count that is
 * a multiple of 8, and 1x1 unpadded windows over (C,H,W) items whose rows the TMA
 * unit can address (C a multiple of 8 and at least 64; unit strides with H*W a
 * multiple of 8, or W a multiple of 8 up to 64 with a column stride of 1 or 2) need
 * none: the kernels read both operands where they are.  Encoded tensor maps are kept per argument list, so a repeated call on the
 * same buffers skips the driver's encoding.  The kernels are launched with programmatic
 * stream serialisation: their set-up may run while the preceding kernel of the stream
 * drains, and they wait for its completion before their first access to memory. */
GL_API int gl_cartesian_dot(const gl_ap* a0, const gl_windows* w_or_null, const gl_ap* a1, gl_ap* out,
                     uint32_t flags, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of scratch gl_cartesian_dot needs for these arguments (0 on invalid ones). */
GL_API size_t gl_cartesian_dot_workspace(const gl_ap* a0, const gl_windows* w_or_null, const gl_ap* a1,
                                  uint32_t flags);

/* gl_cartesian_dot for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a property of the host program, not of the method.)
 *
 * gl_cartesian_dot wants a caller-owned workspace whenever it has to make channels-last
 * copies of its operands.  Code that runs where no allocator may be called - inside
 * another framework's operator, in a plug-in that is handed nothing but its input and
 * output buffers, in a process whose device memory is entirely owned by a pool - cannot
 * provide one.  This variant takes no workspace: it uses a fixed scratch array of
 * GL_STATIC_SCRATCH_BYTES (32 MiB) that is part of the library image, so every GPU that
 * loads the library holds that much memory until the process exits.  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 *   - Same arguments, results and error codes as gl_cartesian_dot without the workspace
 *     pair.  If the layout copies of these arguments exceed GL_STATIC_SCRATCH_BYTES
 *     the call returns GL_ERR_WORKSPACE and launches nothing (for scale: the (C,H,W)
 *     activations of a 32x64x56x56 convolution need 12.3 MiB).  A contraction that
 *     gl_cartesian_dot would split, and whose partial planes do not fit beside the
 *     copies, runs unsplit instead.
 *   - The first call on each device looks up the array's device address (that device
 *     must be current); make that first call before any stream capture begins.
 *   - All calls share the one array and it keeps whatever the last call left in it.
 *     Nothing in it has to start at zero: each call overwrites every byte it later
 *     reads.  Two calls whose kernels can overlap on the GPU (different streams, or
 *     different host threads without ordering) race on the array; order them. */
#define GL_STATIC_SCRATCH_BYTES (32u << 20)
GL_API int gl_cartesian_dot_static(const gl_ap* a0, const gl_windows* w_or_null, const gl_ap* a1, gl_ap* out,
                                   uint32_t flags, void* stream);

/* compute reduceMax (windows? in) (operator table, Fig. 2c max pooling): the largest
 * value of every item; with w given the windows are formed on the fly and never
 * stored.  GL_F32 in any form.  GL_BF16 (results of GL_OUT_BF16 convolutions) in two forms:
 * 2D windows over ((..),(H,W)) items, and channels-last items ((N),(H,W,C)) with window
 * (Kh,Kw,1), stride (Sh,Sw,1) and C a multiple of 8; other bf16 forms return
 * GL_ERR_UNSUPPORTED.  The largest of a set of values is one of them, so nothing is rounded.
 * Inputs must be NaN-free. */
GL_API int gl_compute_reduce_max(const gl_ap* in, const gl_windows* w_or_null, gl_ap* out, void* stream);

/* compute relu (not in the paper's operator table): out = in > 0 ? in : +0, item
 * shape kept.  GL_F32.  in->data == out->data is allowed. */
GL_API int gl_compute_relu(const gl_ap* in, gl_ap* out, void* stream);

/* Synchronises `stream`, then reports and clears the device status word:
 * GL_ERR_TIMEOUT if a bounded wait inside a kernel gave up since the last poll
 * (that kernel's output is then undefined), GL_ERR_CUDA on a runtime error. */
GL_API int gl_poll_device_status(void* stream);

/* Failure-path self-test that faults nothing: launches one block that waits, for at most
 * `limit_ms` (1..1000), on a barrier nothing ever arrives at, using the same bounded wait as the
 * tensor-core pipeline.  The kernel returns normally; the next gl_poll_device_status() on that
 * stream must report GL_ERR_TIMEOUT (and clear it). */
GL_API int gl_selftest_bounded_wait(uint32_t limit_ms, void* stream);

GL_API const char* gl_strerror(int code);
GL_API int gl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GL_H_ */
