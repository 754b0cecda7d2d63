// Internal declarations shared by the translation units of the library.
#pragma once
#include <cstddef>
#include <cstdint>

#include "gl.h"

namespace gl {

inline int64_t prod(const int64_t* s, int lo, int hi) {
  int64_t p = 1;
  for (int i = lo; i < hi; ++i) p *= s[i];
  return p;
}
inline int64_t numel(const gl_ap& a) { return prod(a.shape, 0, a.ndim); }
inline size_t dtype_size(int32_t dt) { return dt == GL_BF16 ? 2 : (dt == GL_F32 ? 4 : 0); }

// Basic well-formedness of an access pattern (shape side only).
int check_meta(const gl_ap* a);
// check_meta plus a non-NULL, 16-byte aligned data pointer.
int check_data(const gl_ap* a);
// out must already carry exactly the inferred metadata.
int check_same_meta(const gl_ap& want, const gl_ap* got);
int check_windows(const gl_ap* in, const gl_windows* w);

// A plain [M,K] x [O,K] -> [M,O] contraction, optionally with the rows of the
// left operand formed on the fly as convolution windows.
struct DotProblem {
  int64_t M = 0, O = 0, K = 0;
  bool conv = false;           // left operand = windows over (C,H,W) or (H,W,C) items
  bool channels_last = false;  // item layout (H,W,C) / (Kh,Kw,C)
  int64_t N = 0, C = 0, H = 0, W = 0, Kh = 0, Kw = 0, Sh = 1, Sw = 1;
  int64_t ph_lo = 0, ph_hi = 0, pw_lo = 0, pw_hi = 0, Ho = 0, Wo = 0;
  bool general = false;        // neither of the above: arbitrary-rank windows
};
int classify_dot(const gl_ap* a0, const gl_windows* w, const gl_ap* a1, DotProblem* p);

}  // namespace gl
