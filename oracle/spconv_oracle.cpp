// CPU oracle for sparse 3D convolution (kernel map + forward).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
// library is checked against.  Nothing in the product path may call it; it shares
// no code, header, table or helper with the CUDA sources.
//
// What it computes (paper sections in brackets):
//   * Sparse tensor = index rows (b, x, y, z) + feature rows [n][C]        [Sec. II-A, data-structure figure]
//   * Location table: coordinate -> input row, here a std::map            [Sec. III-C.1, "Create Location Table"]
//   * Offset table (OFT): for every output row and every kernel offset k the
//     contributing input row or -1                                         [Sec. III-C.2, "Result OFT" figure]
//   * Kernel offset numbering k = kx*K^2 + ky*K + kz                       [Eq. 5]
//   * Strided (regular) convolution: output cell and kernel offset of an
//     input position                                                       [Eq. 1-5, Sec. III-D]
//   * Result: out[o][co] = sum_k sum_c in[OFT[o][k]][c] * w(k, c, co),
//     skipping -1 entries                                                  [Algorithm 2]
//   * Inverse (transposed) convolution: location table on the coarse index set
//     ("indices2"), and for every position of the fine set ("indices1") the related
//     coarse rows with their kernel offsets; the result is again Algorithm 2 over
//     that table                                                           [Sec. III-E]
//
// Readings taken where the paper is silent (each also listed in the design notes):
//   * orientation is correlation: offset k of output cell q looks at input
//     position q*s + d*kvec - pad (the OFT figure puts the (-1,-1) neighbour
//     first and the (+1,+1) neighbour last);
//   * pad = d * floor((K-1)/2); with K == s this gives pad = 0 and Eq. 1-5 exactly;
//   * the batch index is part of the location key (samples never pair);
//   * duplicate input coordinates are an error, not last-writer-wins;
//   * output cells of a strided convolution are all cells touched by at least
//     one input, numbered in lexicographic (b, x, y, z) order; o >= 0 on every axis;
//   * weights are w[k][c][co] (row-major [K^3][Cin][Cout]);
//   * inverse convolution: a fine position p is related to coarse cell q through offset kvec
//     iff p = q*s + d*kvec - pad, i.e. exactly when p feeds q through kvec in the strided
//     convolution with the same parameters; with K == s there is one such pair per fine position
//     (the "singular weight and feature pair" of Sec. III-E), otherwise the related pairs are summed;
//     a fine position without any related coarse row present gets a zero row; the fine rows keep
//     the numbering of the fine index set.
//
// Accumulation is in double; inputs arrive as doubles converted exactly from
// their storage type by the caller.
#include <array>
#include <cstdint>
#include <cstring>
#include <map>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

using Coord = std::array<int32_t, 4>;  // (b, x, y, z); std::array compares lexicographically

struct Kmap {
  int kernel = 0, stride = 0, dilation = 0, submanifold = 0;
  int64_t n_in = 0, n_out = 0, kvol = 0;
  std::vector<Coord> out_coords;                 // [n_out]
  std::vector<int32_t> oft;                      // [n_out][kvol]  input row or -1  (the paper's OFT layout)
  std::vector<std::vector<int32_t>> pair_in;     // per offset k
  std::vector<std::vector<int32_t>> pair_out;    // per offset k
};

inline int floor_half(int K) { return (K - 1) / 2; }

}  // namespace

extern "C" {

// Build the kernel map.  Returns nullptr and sets *err on bad input:
//   1 = invalid argument, 2 = negative coordinate, 3 = duplicate coordinate.
void* oracle_kmap_build(const int32_t* coords, int64_t n, int stride, int dilation, int kernel,
                        int submanifold, int* err) {
  *err = 0;
  if (n < 0 || stride < 1 || dilation < 1 || kernel < 1) { *err = 1; return nullptr; }
  if (submanifold && (stride != 1 || kernel % 2 == 0)) { *err = 1; return nullptr; }
  const int K = kernel, s = stride, d = dilation;
  const int64_t kvol = int64_t(K) * K * K;

  // Location table [Sec. III-C.1]: coordinate -> input row.
  std::map<Coord, int32_t> lct;
  for (int64_t i = 0; i < n; ++i) {
    Coord c{coords[4 * i], coords[4 * i + 1], coords[4 * i + 2], coords[4 * i + 3]};
    for (int a = 0; a < 4; ++a) if (c[a] < 0) { *err = 2; return nullptr; }
    if (!lct.emplace(c, int32_t(i)).second) { *err = 3; return nullptr; }
  }

  auto* km = new Kmap;
  km->kernel = K; km->stride = s; km->dilation = d; km->submanifold = submanifold;
  km->n_in = n; km->kvol = kvol;
  km->pair_in.resize(kvol); km->pair_out.resize(kvol);

  if (submanifold) {
    // Output set = input set, same row numbering [Sec. III-C.2].
    const int r = floor_half(K);
    km->n_out = n;
    km->out_coords.resize(n);
    km->oft.assign(size_t(n) * kvol, -1);
    for (int64_t j = 0; j < n; ++j) {
      Coord c{coords[4 * j], coords[4 * j + 1], coords[4 * j + 2], coords[4 * j + 3]};
      km->out_coords[j] = c;
      for (int kx = 0; kx < K; ++kx)
        for (int ky = 0; ky < K; ++ky)
          for (int kz = 0; kz < K; ++kz) {
            const int64_t k = (int64_t(kx) * K + ky) * K + kz;       // Eq. 5
            Coord q{c[0], c[1] + d * (kx - r), c[2] + d * (ky - r), c[3] + d * (kz - r)};
            auto it = lct.find(q);
            if (it == lct.end()) continue;
            km->oft[size_t(j) * kvol + k] = it->second;
            km->pair_in[k].push_back(it->second);
            km->pair_out[k].push_back(int32_t(j));
          }
    }
    return km;
  }

  // Regular / strided convolution [Sec. III-D].  An input at position p feeds
  // output cell o through offset kvec iff p = o*s + d*kvec - pad, o >= 0.
  const int pad = d * floor_half(K);
  std::map<Coord, int32_t> outs;  // first pass: which cells are touched
  for (int64_t i = 0; i < n; ++i) {
    const int32_t* p = coords + 4 * i;
    for (int kx = 0; kx < K; ++kx)
      for (int ky = 0; ky < K; ++ky)
        for (int kz = 0; kz < K; ++kz) {
          const int kv[3] = {kx, ky, kz};
          Coord o{p[0], 0, 0, 0};
          bool ok = true;
          for (int a = 0; a < 3 && ok; ++a) {
            const int num = p[a + 1] + pad - d * kv[a];
            if (num < 0 || num % s != 0) ok = false; else o[a + 1] = num / s;
          }
          if (ok) outs.emplace(o, 0);
        }
  }
  // Number the touched cells in map (lexicographic) order.
  km->n_out = int64_t(outs.size());
  km->out_coords.reserve(outs.size());
  { int32_t idx = 0; for (auto& kv : outs) { kv.second = idx++; km->out_coords.push_back(kv.first); } }
  km->oft.assign(size_t(km->n_out) * kvol, -1);
  // Second pass: for every output cell and offset consult the location table.
  for (int64_t o = 0; o < km->n_out; ++o) {
    const Coord& q = km->out_coords[o];
    for (int kx = 0; kx < K; ++kx)
      for (int ky = 0; ky < K; ++ky)
        for (int kz = 0; kz < K; ++kz) {
          const int64_t k = (int64_t(kx) * K + ky) * K + kz;
          Coord p{q[0], q[1] * s + d * kx - pad, q[2] * s + d * ky - pad, q[3] * s + d * kz - pad};
          auto it = lct.find(p);
          if (it == lct.end()) continue;
          km->oft[size_t(o) * kvol + k] = it->second;
          km->pair_in[k].push_back(it->second);
          km->pair_out[k].push_back(int32_t(o));
        }
  }
  return km;
}

// Kernel map of the inverse convolution [Sec. III-E].  Stage 1: location table over the coarse
// index set (fine -> "indices1" [n_fine][4], coarse -> "indices2" [n_coarse][4] in the paper's
// words).  Stage 2: every fine position, every kernel offset: which coarse row is related through
// that offset.  The returned map has n_in = n_coarse (rows of the input features), n_out = n_fine
// (output row j = fine row j); its OFT row j lists, per offset k, the coarse row or -1.
// Errors as for oracle_kmap_build (duplicates are checked in both sets).
void* oracle_inverse_kmap_build(const int32_t* fine, int64_t n_fine, const int32_t* coarse, int64_t n_coarse,
                                int stride, int dilation, int kernel, int* err) {
  *err = 0;
  if (n_fine < 0 || n_coarse < 0 || stride < 1 || dilation < 1 || kernel < 1) { *err = 1; return nullptr; }
  const int K = kernel, s = stride, d = dilation;
  const int64_t kvol = int64_t(K) * K * K;
  const int pad = d * floor_half(K);

  std::map<Coord, int32_t> lct2;   // location table of the coarse set
  for (int64_t i = 0; i < n_coarse; ++i) {
    Coord c{coarse[4 * i], coarse[4 * i + 1], coarse[4 * i + 2], coarse[4 * i + 3]};
    for (int a = 0; a < 4; ++a) if (c[a] < 0) { *err = 2; return nullptr; }
    if (!lct2.emplace(c, int32_t(i)).second) { *err = 3; return nullptr; }
  }
  {
    std::map<Coord, int32_t> seen;
    for (int64_t j = 0; j < n_fine; ++j) {
      Coord c{fine[4 * j], fine[4 * j + 1], fine[4 * j + 2], fine[4 * j + 3]};
      for (int a = 0; a < 4; ++a) if (c[a] < 0) { *err = 2; return nullptr; }
      if (!seen.emplace(c, int32_t(j)).second) { *err = 3; return nullptr; }
    }
  }

  auto* km = new Kmap;
  km->kernel = K; km->stride = s; km->dilation = d; km->submanifold = 0;
  km->n_in = n_coarse; km->n_out = n_fine; km->kvol = kvol;
  km->pair_in.resize(kvol); km->pair_out.resize(kvol);
  km->out_coords.resize(n_fine);
  km->oft.assign(size_t(n_fine) * kvol, -1);
  for (int64_t j = 0; j < n_fine; ++j) {
    const int32_t* p = fine + 4 * j;
    km->out_coords[j] = Coord{p[0], p[1], p[2], p[3]};
    for (int kx = 0; kx < K; ++kx)
      for (int ky = 0; ky < K; ++ky)
        for (int kz = 0; kz < K; ++kz) {
          const int64_t k = (int64_t(kx) * K + ky) * K + kz;       // Eq. 5
          const int kv[3] = {kx, ky, kz};
          Coord q{p[0], 0, 0, 0};
          bool ok = true;
          for (int a = 0; a < 3 && ok; ++a) {
            const int num = p[a + 1] + pad - d * kv[a];              // q*s = p + pad - d*kvec
            if (num < 0 || num % s != 0) ok = false; else q[a + 1] = num / s;
          }
          if (!ok) continue;
          auto it = lct2.find(q);
          if (it == lct2.end()) continue;
          km->oft[size_t(j) * kvol + k] = it->second;
          km->pair_in[k].push_back(it->second);
          km->pair_out[k].push_back(int32_t(j));
        }
  }
  return km;
}

int64_t oracle_kmap_n_out(const void* h) { return static_cast<const Kmap*>(h)->n_out; }
int64_t oracle_kmap_kvol(const void* h) { return static_cast<const Kmap*>(h)->kvol; }
int64_t oracle_kmap_total_pairs(const void* h) {
  int64_t p = 0; for (auto& v : static_cast<const Kmap*>(h)->pair_in) p += int64_t(v.size()); return p;
}

// Copy the tables out.  out_coords [n_out][4]; oft [n_out][kvol]; offset_start [kvol+1];
// pair_in / pair_out [total_pairs], offset k occupying [offset_start[k], offset_start[k+1]).
void oracle_kmap_export(const void* h, int32_t* out_coords, int32_t* oft, int64_t* offset_start,
                        int32_t* pair_in, int32_t* pair_out) {
  const Kmap* km = static_cast<const Kmap*>(h);
  for (int64_t o = 0; o < km->n_out; ++o) for (int a = 0; a < 4; ++a) out_coords[4 * o + a] = km->out_coords[o][a];
  if (!km->oft.empty()) std::memcpy(oft, km->oft.data(), km->oft.size() * sizeof(int32_t));
  int64_t pos = 0;
  for (int64_t k = 0; k < km->kvol; ++k) {
    offset_start[k] = pos;
    for (size_t t = 0; t < km->pair_in[k].size(); ++t) { pair_in[pos] = km->pair_in[k][t]; pair_out[pos] = km->pair_out[k][t]; ++pos; }
  }
  offset_start[km->kvol] = pos;
}

void oracle_kmap_free(void* h) { delete static_cast<Kmap*>(h); }

// Forward result per Algorithm 2 over an OFT [n_out][kvol]:
//   out[i][o] = sum_k [oft[i][k] != -1] sum_c feats[oft[i][k]][c] * w[k][c][o]
// feats [n_in][cin], w [kvol][cin][cout], out [n_out][cout]; all double.
// Rows are independent; the loop over rows is the only parallel loop.
void oracle_forward(const double* feats, const double* w, const int32_t* oft, int64_t n_out, int64_t kvol,
                    int cin, int cout, double* out) {
#pragma omp parallel for schedule(dynamic, 64)
  for (int64_t i = 0; i < n_out; ++i) {
    for (int o = 0; o < cout; ++o) {
      double s = 0.0;
      for (int64_t k = 0; k < kvol; ++k) {
        const int32_t nidx = oft[i * kvol + k];
        if (nidx == -1) continue;
        for (int c = 0; c < cin; ++c) s += feats[int64_t(nidx) * cin + c] * w[(k * cin + c) * cout + o];
      }
      out[i * cout + o] = s;
    }
  }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
