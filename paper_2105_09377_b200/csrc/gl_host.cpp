// Host-only part of the library: argument validation and the shape rules of
// the access-pattern transformers (Section 4.2, transformer table) and of
// `compute` (Section 4.3).  Nothing here touches the device.
#include <cstring>

#include "gl_internal.h"

namespace gl {

int check_meta(const gl_ap* a) {
  if (!a) return GL_ERR_NULL;
  if (a->dtype != GL_BF16 && a->dtype != GL_F32) return GL_ERR_DTYPE;
  if (a->ndim < 0 || a->ndim > GL_MAX_DIMS) return GL_ERR_NDIM;
  if (a->access_ndim < 0 || a->access_ndim > a->ndim) return GL_ERR_NDIM;
  for (int i = 0; i < a->ndim; ++i)
    if (a->shape[i] < 1) return GL_ERR_SHAPE;  // shapes are tuples of positive integers
  return GL_OK;
}

int check_data(const gl_ap* a) {
  int rc = check_meta(a);
  if (rc) return rc;
  if (!a->data) return GL_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(a->data) & 15u) return GL_ERR_ALIGN;
  return GL_OK;
}

int check_same_meta(const gl_ap& want, const gl_ap* got) {
  if (!got) return GL_ERR_NULL;
  if (got->dtype != want.dtype) return GL_ERR_DTYPE;
  if (got->ndim != want.ndim || got->access_ndim != want.access_ndim) return GL_ERR_SHAPE;
  for (int i = 0; i < want.ndim; ++i)
    if (got->shape[i] != want.shape[i]) return GL_ERR_SHAPE;
  return GL_OK;
}

int check_windows(const gl_ap* in, const gl_windows* w) {
  if (!w) return GL_ERR_NULL;
  const int n = in->ndim - in->access_ndim;
  if (w->n != n) return GL_ERR_SHAPE;  // one extent and stride per compute dimension
  if (w->pad_kind != GL_PAD_ZERO && w->pad_kind != GL_PAD_NEG_INF) return GL_ERR_SHAPE;
  if (in->access_ndim + 2 * n > GL_MAX_DIMS) return GL_ERR_NDIM;
  for (int i = 0; i < n; ++i) {
    const int64_t b = in->shape[in->access_ndim + i];
    if (w->wshape[i] < 1 || w->stride[i] < 1) return GL_ERR_SHAPE;
    if (w->pad_lo[i] < 0 || w->pad_hi[i] < 0) return GL_ERR_SHAPE;
    // every window must hold at least one real cell
    if (w->pad_lo[i] >= w->wshape[i] || w->pad_hi[i] >= w->wshape[i]) return GL_ERR_SHAPE;
    if (w->wshape[i] > b + w->pad_lo[i] + w->pad_hi[i]) return GL_ERR_SHAPE;
  }
  return GL_OK;
}

static void copy_meta(const gl_ap* in, gl_ap* out) {
  void* keep = out->data;
  *out = *in;
  out->data = keep;
}

// b' = ceil((b - (w - 1)) / s) on the padded extent (transformer table, `windows`).
static int64_t windows_extent(int64_t b, int64_t w, int64_t s) { return (b - (w - 1) + s - 1) / s; }

static int infer_windows(const gl_ap* in, const gl_windows* w, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  rc = check_windows(in, w);
  if (rc) return rc;
  const int na = in->access_ndim, n = w->n;
  gl_ap r;
  std::memset(&r, 0, sizeof(r));
  r.dtype = in->dtype;
  r.ndim = na + 2 * n;
  r.access_ndim = na + n;
  for (int i = 0; i < na; ++i) r.shape[i] = in->shape[i];
  for (int i = 0; i < n; ++i) {
    const int64_t b = in->shape[na + i] + w->pad_lo[i] + w->pad_hi[i];
    r.shape[na + i] = windows_extent(b, w->wshape[i], w->stride[i]);
    r.shape[na + n + i] = w->wshape[i];
  }
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int classify_dot(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, DotProblem* p) {
  int rc = check_meta(a0);
  if (rc) return rc;
  rc = check_meta(a1);
  if (rc) return rc;
  gl_ap A = *a0;
  if (w) {
    rc = infer_windows(a0, w, &A);
    if (rc) return rc;
  }
  // cartProd needs equal compute shapes (transformer table)
  const int nk = A.ndim - A.access_ndim;
  if (nk != a1->ndim - a1->access_ndim) return GL_ERR_SHAPE;
  for (int i = 0; i < nk; ++i)
    if (A.shape[A.access_ndim + i] != a1->shape[a1->access_ndim + i]) return GL_ERR_SHAPE;
  if (A.access_ndim + a1->access_ndim > GL_MAX_DIMS) return GL_ERR_NDIM;
  DotProblem d;
  d.M = prod(A.shape, 0, A.access_ndim);
  d.K = prod(A.shape, A.access_ndim, A.ndim);
  d.O = prod(a1->shape, 0, a1->access_ndim);
  if (w) {
    const int na = a0->access_ndim;
    const int64_t* b = a0->shape + na;
    bool nchw = w->n == 3 && w->wshape[0] == b[0] && w->pad_lo[0] == 0 && w->pad_hi[0] == 0;
    bool nhwc = w->n == 3 && w->wshape[2] == b[2] && w->pad_lo[2] == 0 && w->pad_hi[2] == 0;
    if (w->pad_kind != GL_PAD_ZERO) nchw = nhwc = false;
    if (nchw || nhwc) {
      d.conv = true;
      d.channels_last = !nchw;
      const int ih = nchw ? 1 : 0, iw = nchw ? 2 : 1, ic = nchw ? 0 : 2;
      d.N = prod(a0->shape, 0, na);
      d.C = b[ic]; d.H = b[ih]; d.W = b[iw];
      d.Kh = w->wshape[ih]; d.Kw = w->wshape[iw];
      d.Sh = w->stride[ih]; d.Sw = w->stride[iw];
      d.ph_lo = w->pad_lo[ih]; d.ph_hi = w->pad_hi[ih];
      d.pw_lo = w->pad_lo[iw]; d.pw_hi = w->pad_hi[iw];
      d.Ho = A.shape[na + ih]; d.Wo = A.shape[na + iw];
    } else {
      d.general = true;
    }
  }
  *p = d;
  return GL_OK;
}

}  // namespace gl

using namespace gl;

extern "C" {

int gl_shape_access(const gl_ap* in, int32_t i, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (i < 0 || i > in->ndim) return GL_ERR_NDIM;
  copy_meta(in, out);
  out->access_ndim = i;
  return GL_OK;
}

int gl_shape_windows(const gl_ap* in, const gl_windows* w, gl_ap* out) {
  if (!out) return GL_ERR_NULL;
  return infer_windows(in, w, out);
}

int gl_shape_flatten(const gl_ap* in, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  gl_ap r;
  std::memset(&r, 0, sizeof(r));
  r.dtype = in->dtype;
  const int na = in->access_ndim, nc = in->ndim - na;
  if (na) r.shape[r.ndim++] = prod(in->shape, 0, na);
  r.access_ndim = r.ndim;
  if (nc) r.shape[r.ndim++] = prod(in->shape, na, in->ndim);
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_transpose(const gl_ap* in, const int32_t* perm, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!perm || !out) return GL_ERR_NULL;
  bool seen[GL_MAX_DIMS] = {false};
  for (int i = 0; i < in->ndim; ++i) {
    if (perm[i] < 0 || perm[i] >= in->ndim || seen[perm[i]]) return GL_ERR_PERM;
    seen[perm[i]] = true;
  }
  gl_ap r = *in;
  for (int i = 0; i < in->ndim; ++i) r.shape[i] = in->shape[perm[i]];
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_pad(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (dim < 0 || dim >= in->ndim) return GL_ERR_NDIM;
  if (lo < 0 || hi < 0) return GL_ERR_SHAPE;
  copy_meta(in, out);
  out->shape[dim] += lo + hi;
  return GL_OK;
}

int gl_shape_slice(const gl_ap* in, int32_t dim, int64_t lo, int64_t hi, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (dim < 0 || dim >= in->ndim) return GL_ERR_NDIM;
  if (lo < 0 || hi <= lo || hi > in->shape[dim]) return GL_ERR_SHAPE;
  copy_meta(in, out);
  out->shape[dim] = hi - lo;
  return GL_OK;
}

int gl_shape_concat(const gl_ap* a, const gl_ap* b, int32_t dim, gl_ap* out) {
  int rc = check_meta(a);
  if (rc) return rc;
  rc = check_meta(b);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (a->dtype != b->dtype) return GL_ERR_DTYPE;
  if (dim < 0 || dim >= a->ndim) return GL_ERR_NDIM;
  if (a->ndim != b->ndim || a->access_ndim != b->access_ndim) return GL_ERR_SHAPE;
  for (int i = 0; i < a->ndim; ++i)
    if (i != dim && a->shape[i] != b->shape[i]) return GL_ERR_SHAPE;
  copy_meta(a, out);
  out->shape[dim] = a->shape[dim] + b->shape[dim];
  return GL_OK;
}

int gl_shape_pair(const gl_ap* a, const gl_ap* b, gl_ap* out) {
  int rc = check_meta(a);
  if (rc) return rc;
  rc = check_meta(b);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (a->dtype != b->dtype) return GL_ERR_DTYPE;
  if (a->ndim + 1 > GL_MAX_DIMS) return GL_ERR_NDIM;
  if (a->ndim != b->ndim || a->access_ndim != b->access_ndim) return GL_ERR_SHAPE;
  for (int i = 0; i < a->ndim; ++i)
    if (a->shape[i] != b->shape[i]) return GL_ERR_SHAPE;
  gl_ap r = *a;
  r.ndim = a->ndim + 1;
  r.shape[a->access_ndim] = 2;   // the 2 is the first compute dimension
  for (int i = a->access_ndim; i < a->ndim; ++i) r.shape[i + 1] = a->shape[i];
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_squeeze(const gl_ap* in, int32_t dim, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  if (dim < 0 || dim >= in->ndim) return GL_ERR_NDIM;
  if (in->shape[dim] != 1) return GL_ERR_SHAPE;
  gl_ap r = *in;
  for (int i = dim; i + 1 < in->ndim; ++i) r.shape[i] = in->shape[i + 1];
  r.shape[in->ndim - 1] = 0;
  r.ndim = in->ndim - 1;
  if (dim < in->access_ndim) r.access_ndim = in->access_ndim - 1;
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_reshape(const gl_ap* in, const int64_t* shape, int32_t ndim, int32_t access_ndim, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out || (!shape && ndim > 0)) return GL_ERR_NULL;
  if (ndim < 0 || ndim > GL_MAX_DIMS || access_ndim < 0 || access_ndim > ndim) return GL_ERR_NDIM;
  for (int i = 0; i < ndim; ++i)
    if (shape[i] < 1) return GL_ERR_SHAPE;
  if (prod(shape, 0, access_ndim) != prod(in->shape, 0, in->access_ndim)) return GL_ERR_SHAPE;
  if (prod(shape, access_ndim, ndim) != prod(in->shape, in->access_ndim, in->ndim)) return GL_ERR_SHAPE;
  gl_ap r;
  std::memset(&r, 0, sizeof(r));
  r.dtype = in->dtype;
  r.ndim = ndim;
  r.access_ndim = access_ndim;
  for (int i = 0; i < ndim; ++i) r.shape[i] = shape[i];
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_reduce_sum(const gl_ap* in, gl_ap* out) { return gl_shape_reduce_max(in, nullptr, out); }

int gl_shape_cartesian_dot(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, gl_ap* out) {
  if (!out) return GL_ERR_NULL;
  DotProblem d;
  int rc = classify_dot(a0, w, a1, &d);
  if (rc) return rc;
  gl_ap A = *a0;
  if (w) infer_windows(a0, w, &A);
  gl_ap r;
  std::memset(&r, 0, sizeof(r));
  r.dtype = GL_F32;
  for (int i = 0; i < A.access_ndim; ++i) r.shape[r.ndim++] = A.shape[i];
  for (int i = 0; i < a1->access_ndim; ++i) r.shape[r.ndim++] = a1->shape[i];
  r.access_ndim = r.ndim;
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_cartesian_dot_nchw(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, gl_ap* out) {
  if (!out) return GL_ERR_NULL;
  if (!w) return GL_ERR_SHAPE;
  DotProblem d;
  int rc = classify_dot(a0, w, a1, &d);
  if (rc) return rc;
  if (!d.conv) return GL_ERR_UNSUPPORTED;   // only the conv2d item layouts have an H' and a W'
  if (a0->access_ndim + a1->access_ndim + 2 > GL_MAX_DIMS) return GL_ERR_NDIM;
  gl_ap r;
  std::memset(&r, 0, sizeof(r));
  r.dtype = GL_F32;
  for (int i = 0; i < a0->access_ndim; ++i) r.shape[r.ndim++] = a0->shape[i];
  for (int i = 0; i < a1->access_ndim; ++i) r.shape[r.ndim++] = a1->shape[i];
  r.shape[r.ndim++] = d.Ho;
  r.shape[r.ndim++] = d.Wo;
  r.access_ndim = r.ndim;
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_shape_reduce_max(const gl_ap* in, const gl_windows* w, gl_ap* out) {
  if (!out) return GL_ERR_NULL;
  int rc = check_meta(in);
  if (rc) return rc;
  gl_ap A = *in;
  if (w) {
    rc = infer_windows(in, w, &A);
    if (rc) return rc;
  }
  if (A.ndim == A.access_ndim) return GL_ERR_SHAPE;  // nothing to reduce
  gl_ap r = A;
  r.ndim = A.access_ndim;
  for (int i = r.ndim; i < GL_MAX_DIMS; ++i) r.shape[i] = 0;
  r.data = out->data;
  *out = r;
  return GL_OK;
}

int gl_access_flatten(const gl_ap* in, gl_ap* out) {
  int rc = check_meta(in);
  if (rc) return rc;
  if (!out) return GL_ERR_NULL;
  rc = gl_shape_flatten(in, out);
  if (rc) return rc;
  out->data = in->data;
  return GL_OK;
}

const char* gl_strerror(int code) {
  switch (code) {
    case GL_OK: return "ok";
    case GL_ERR_NULL: return "a required pointer is NULL";
    case GL_ERR_DTYPE: return "dtype not accepted by this call";
    case GL_ERR_NDIM: return "ndim or access_ndim out of range";
    case GL_ERR_SHAPE: return "shapes disagree";
    case GL_ERR_PERM: return "not a permutation of the dimensions";
    case GL_ERR_ALIGN: return "data pointer not 16-byte aligned";
    case GL_ERR_UNSUPPORTED: return "no kernel covers this combination";
    case GL_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case GL_ERR_CUDA: return "CUDA error";
    case GL_ERR_TIMEOUT: return "a bounded wait inside a kernel gave up";
    default: return "unknown error code";
  }
}

int gl_version(void) { return 100; }

}  // extern "C"
