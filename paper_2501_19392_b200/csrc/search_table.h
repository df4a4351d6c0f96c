// Host-side construction of the cell table that prunes the nearest-grid-point search of the
// backbone quantizer (Section 2 "Vector Quantization": every pair of rotated values is rounded to
// the nearest of n fixed 2-D points; Section 4.1: n in {16, 64, 256}).
//
// The square [-B, B)^2 is cut into C x C cells.  For each cell the table lists every grid point
// whose Voronoi region meets the (slightly inflated) cell, so the exact arg-min over ALL points
// equals the arg-min over the listed ones for any y inside the cell.  Cells that need more
// candidates than the kernel evaluates in its fast path (three for n = 16, four for larger grids)
// are searched exhaustively by the kernel, and so are values outside the square; for n > 64, where
// such cells are common, those with at most eight candidates point to a second-level list of eight
// instead.  The table therefore never changes a result,
// it only skips points that cannot win.
//
// Entry layout (uint32): bytes 3, 2, 1, 0 = candidate indices in ascending order (byte 3 the
// lowest; short lists repeat their last index), so every plain entry is below 0xFF000000 unless
// its only candidate is point 255.  0xFF000000 + i points to second-level list i (two uint32 after
// the cells: eight ascending candidates, byte 0 of the first word the lowest, short lists repeat
// their last index).  0xFFFFFFFF marks a cell that must be searched exhaustively, which includes
// all border cells: the kernel clamps cell coordinates, so they stand for everything outside the
// square.  The kernel finds the special entries with one unsigned comparison.
#pragma once

#include <cmath>
#include <cstdint>
#include <vector>

namespace aquakv {

constexpr uint32_t kCellBrute = 0xFFFFFFFFu;   // the largest entry value; as a candidate list it could only
                                               // mean "point 255 alone", for which searching all points is right too
constexpr uint32_t kCellSpecial = 0xFF000000u; // entries >= this are second-level references or kCellBrute
constexpr int kSearchMaxLists = 2048;          // second-level lists the table has room for
constexpr int kSearchListLen = 8;

struct SearchTableSpec {
  int cells;        // C, cells per side (power of two)
  int log_cells;
  float half;       // B
  float inv_w;      // C / (2B), the value the kernel multiplies by
  int max_cand;     // candidates the kernel evaluates per pair
};

inline SearchTableSpec search_table_spec(const float* grid, int n) {
  float m = 0.0f;
  for (int i = 0; i < 2 * n; ++i) m = std::fmax(m, std::fabs(grid[i]));
  SearchTableSpec s;
  s.max_cand = n <= 16 ? 3 : 4;
  s.cells = 64;          // kSearchCells of codec.cuh: the kernels keep the table in shared memory
  s.log_cells = 6;
  s.half = std::ceil((m + 2.0f) * 4.0f) / 4.0f;
  s.inv_w = float(s.cells) / (2.0f * s.half);
  return s;
}

namespace detail {
struct Pt { double x, y; };

// Keeps the part of the convex polygon with a.x*x + a.y*y <= b (Sutherland-Hodgman).
inline void clip(std::vector<Pt>& poly, double ax, double ay, double b) {
  std::vector<Pt> out;
  const size_t m = poly.size();
  for (size_t i = 0; i < m; ++i) {
    const Pt p = poly[i], q = poly[(i + 1) % m];
    const double fp = ax * p.x + ay * p.y - b, fq = ax * q.x + ay * q.y - b;
    if (fp <= 0.0) out.push_back(p);
    if ((fp < 0.0 && fq > 0.0) || (fp > 0.0 && fq < 0.0)) {
      const double t = fp / (fp - fq);
      out.push_back(Pt{p.x + t * (q.x - p.x), p.y + t * (q.y - p.y)});
    }
  }
  poly.swap(out);
}
}  // namespace detail

// Words of a table buffer: the cells followed by the second-level lists (two words each).
inline size_t search_table_words(const SearchTableSpec& s) {
  return size_t(s.cells) * s.cells + size_t(2) * kSearchMaxLists;
}

// Fills table[cells*cells] (row = y cell, column = x cell) and the second-level lists behind it;
// returns the number of lists used (the rest of the buffer is zeroed).
inline int build_search_table(const float* grid, int n, const SearchTableSpec& s, uint32_t* table) {
  const int C = s.cells;
  const double w = 1.0 / double(s.inv_w);
  const double eps = 1e-3 * w + 1e-5;        // covers fp32 rounding of the cell index and scores
  const double tol = 1e-9;
  std::vector<double> dist(n);
  std::vector<int> pre, cand;
  std::vector<detail::Pt> poly;
  uint32_t* lists = table + size_t(C) * C;
  for (int i = 0; i < 2 * kSearchMaxLists; ++i) lists[i] = 0;
  int n_lists = 0;
  for (int iy = 0; iy < C; ++iy) {
    for (int ix = 0; ix < C; ++ix) {
      const double x0 = (ix - C / 2) * w - eps, x1 = (ix + 1 - C / 2) * w + eps;
      const double y0 = (iy - C / 2) * w - eps, y1 = (iy + 1 - C / 2) * w + eps;
      const double cx = 0.5 * (x0 + x1), cy = 0.5 * (y0 + y1);
      const double r = 0.5 * std::sqrt((x1 - x0) * (x1 - x0) + (y1 - y0) * (y1 - y0));
      double dmin = 1e300;
      for (int j = 0; j < n; ++j) {
        const double dx = cx - grid[2 * j], dy = cy - grid[2 * j + 1];
        dist[j] = std::sqrt(dx * dx + dy * dy);
        dmin = std::fmin(dmin, dist[j]);
      }
      // a point farther than dmin + 2r from the centre loses everywhere in the cell
      pre.clear();
      for (int j = 0; j < n; ++j)
        if (dist[j] <= dmin + 2.0 * r + 1e-9) pre.push_back(j);
      cand.clear();
      for (int i : pre) {
        poly.assign({{x0, y0}, {x1, y0}, {x1, y1}, {x0, y1}});
        const double gix = grid[2 * i], giy = grid[2 * i + 1];
        for (int k : pre) {
          if (k == i || poly.empty()) continue;
          const double gkx = grid[2 * k], gky = grid[2 * k + 1];
          // |y - g_i|^2 <= |y - g_k|^2   <=>   2 y.(g_k - g_i) <= |g_k|^2 - |g_i|^2
          detail::clip(poly, 2.0 * (gkx - gix), 2.0 * (gky - giy),
                       gkx * gkx + gky * gky - gix * gix - giy * giy + tol);
        }
        if (!poly.empty()) cand.push_back(i);
      }
      uint32_t e;
      // border cells also catch every value outside the square (the kernel's cell index saturates)
      const bool border = ix == 0 || iy == 0 || ix == C - 1 || iy == C - 1;
      const int nc = int(cand.size());
      auto at = [&](int k) { return uint32_t(cand[k < nc ? k : nc - 1]); };
      const bool may_list = n > 64 && nc <= kSearchListLen && n_lists < kSearchMaxLists;
      if (border || cand.empty() || (nc > s.max_cand && !may_list)) {
        e = kCellBrute;
      } else if (nc > s.max_cand) {
        e = kCellSpecial + uint32_t(n_lists);
        for (int k = 0; k < 4; ++k) {
          lists[2 * n_lists] |= at(k) << (8 * k);
          lists[2 * n_lists + 1] |= at(4 + k) << (8 * k);
        }
        ++n_lists;
      } else {
        e = 0;
        for (int k = 0; k < 4; ++k) e |= at(k) << (8 * (3 - k));
      }
      table[size_t(iy) * C + ix] = e;
    }
  }
  return n_lists;
}

}  // namespace aquakv
