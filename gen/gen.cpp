// Seeded synthetic workload generators (host only, no CUDA, none of the SpMV/SpMM arithmetic).
//
// These produce the CSR matrices and dense operands that both the CPU oracle's tests and the
// GPU path's tests and benchmark consume.  Every sample comes from a counter-based hash of
// (seed, stream, index), so results do not depend on thread count or evaluation order.
//
// Workload shapes follow the sparse-matrix task class of the paper's benchmark (Appendix C,
// Table 6, tasks 12 and 13: CSR arrays values / col_indices / row_offsets) at the sizes this
// project measures: a 2D 5-point Laplacian, fixed-nnz-per-row uniform matrices, an R-MAT
// power-law graph and a 3D 27-point stencil.
#include <cstdint>
#include <cstring>
#include <cmath>
#include <vector>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#include <parallel/algorithm>
#endif

namespace {

inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
// Counter-based generator: one 64-bit word per (seed, stream, index).
inline uint64_t rnd(uint64_t seed, uint64_t stream, uint64_t idx) {
  uint64_t k = mix64(seed * 0x9E3779B97F4A7C15ull + stream * 0xD1B54A32D192ED03ull + 0x632BE59BD9B4E019ull);
  return mix64(k + idx * 0x9E3779B97F4A7C15ull);
}
inline float u01(uint64_t h) { return (float)(h >> 40) * (1.0f / 16777216.0f); }             // [0,1), 24 bits
inline float u01_open_low(uint64_t h) { return (float)((h >> 40) + 1) * (1.0f / 16777216.0f); } // (0,1]
inline double normal01(uint64_t seed, uint64_t stream, uint64_t idx) {
  const double u1 = (double)((rnd(seed, stream, 2 * idx) >> 11) + 1) * (1.0 / 9007199254740992.0);  // (0,1]
  const double u2 = (double)(rnd(seed, stream, 2 * idx + 1) >> 11) * (1.0 / 9007199254740992.0);    // [0,1)
  return std::sqrt(-2.0 * std::log(u1)) * std::cos(6.283185307179586476925 * u2);
}
inline uint32_t bounded(uint64_t h, uint32_t n) { return (uint32_t)(((h >> 32) * (uint64_t)n) >> 32); }

}  // namespace

extern "C" {

// ---------------------------------------------------------------- dense operands
void gen_uniform(int64_t n, float lo, float hi, uint64_t seed, uint64_t stream, float* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = lo + (hi - lo) * u01(rnd(seed, stream, (uint64_t)i));
}
void gen_uniform_open_low(int64_t n, uint64_t seed, uint64_t stream, float* out) {  // (0,1]
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = u01_open_low(rnd(seed, stream, (uint64_t)i));
}
void gen_normal(int64_t n, float mean, float sigma, uint64_t seed, uint64_t stream, float* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = (float)((double)mean + (double)sigma * normal01(seed, stream, (uint64_t)i));
}
// Storage conversion FP32 -> BF16 bit pattern, round to nearest even (inputs are finite).
void gen_f32_to_bf16(int64_t n, const float* in, uint16_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    uint32_t u; std::memcpy(&u, &in[i], 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    out[i] = (uint16_t)(u >> 16);
  }
}

// ---------------------------------------------------------------- 2D 5-point Laplacian
// Grid N x N, row index i*N + j, diagonal 4, existing neighbours -1 (neighbours outside the grid dropped).
int64_t gen_lap2d_nnz(int64_t N) { return 5 * N * N - 4 * N; }
void gen_lap2d(int64_t N, int32_t* row_ptr, int32_t* col_idx, float* vals) {
  int64_t p = 0;
  for (int64_t i = 0; i < N; ++i)
    for (int64_t j = 0; j < N; ++j) {
      const int64_t r = i * N + j;
      row_ptr[r] = (int32_t)p;
      if (i > 0)     { col_idx[p] = (int32_t)(r - N); vals[p++] = -1.0f; }
      if (j > 0)     { col_idx[p] = (int32_t)(r - 1); vals[p++] = -1.0f; }
      col_idx[p] = (int32_t)r; vals[p++] = 4.0f;
      if (j < N - 1) { col_idx[p] = (int32_t)(r + 1); vals[p++] = -1.0f; }
      if (i < N - 1) { col_idx[p] = (int32_t)(r + N); vals[p++] = -1.0f; }
    }
  row_ptr[N * N] = (int32_t)p;
}

// ---------------------------------------------------------------- fixed nnz per row, uniform columns
// Each row: per_row iid uniform columns, sorted; the whole row is redrawn while it holds a duplicate
// (uniform over per_row-subsets).  Values N(0,1).
void gen_uniform_rows(int64_t m, int64_t n, int32_t per_row, uint64_t seed,
                      int32_t* row_ptr, int32_t* col_idx, float* vals) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < m; ++i) {
    int32_t* c = col_idx + i * per_row;
    for (uint64_t attempt = 0;; ++attempt) {
      for (int32_t j = 0; j < per_row; ++j)
        c[j] = (int32_t)bounded(rnd(seed, 100 + attempt, (uint64_t)(i * per_row + j)), (uint32_t)n);
      std::sort(c, c + per_row);
      bool dup = false;
      for (int32_t j = 1; j < per_row; ++j) dup |= (c[j] == c[j - 1]);
      if (!dup) break;
    }
    row_ptr[i] = (int32_t)(i * per_row);
    for (int32_t j = 0; j < per_row; ++j)
      vals[i * per_row + j] = (float)normal01(seed, 1, (uint64_t)(i * per_row + j));
  }
  row_ptr[m] = (int32_t)(m * per_row);
}

// ---------------------------------------------------------------- R-MAT power-law graph
// 2^scale vertices; e_gen directed edges drawn by recursive quadrant choice with probabilities
// (a, b, c, 1-a-b-c) per level; no noise, no relabelling, self loops kept; sorted by (row, col),
// duplicates dropped.  Returns nnz after dedup; the caller passes buffers of e_gen entries.
// Values uniform (0,1].
// A bijection of [0, 2^scale): two rounds of xor-shift and an odd multiply-add, each invertible mod 2^scale.
static inline uint32_t relabel_vertex(uint32_t v, int32_t scale, uint64_t seed) {
  const uint32_t mask = scale >= 32 ? 0xFFFFFFFFu : ((1u << scale) - 1u);
  const int32_t sh = scale / 2 > 0 ? scale / 2 : 1;
  const uint32_t m1 = ((uint32_t)rnd(seed, 300, 0) | 1u), m2 = ((uint32_t)rnd(seed, 300, 1) | 1u);
  const uint32_t c1 = (uint32_t)(rnd(seed, 300, 2)), c2 = (uint32_t)(rnd(seed, 300, 3));
  v ^= v >> sh; v = (v * m1 + c1) & mask;
  v ^= v >> sh; v = (v * m2 + c2) & mask;
  v ^= v >> sh;
  return v;
}

static int64_t gen_rmat_impl(int32_t scale, int64_t e_gen, double a, double b, double c, uint64_t seed, bool relabel,
                             int32_t* row_ptr, int32_t* col_idx, float* vals);

int64_t gen_rmat(int32_t scale, int64_t e_gen, double a, double b, double c, uint64_t seed,
                 int32_t* row_ptr, int32_t* col_idx, float* vals) {
  return gen_rmat_impl(scale, e_gen, a, b, c, seed, false, row_ptr, col_idx, vals);
}

// Same edges with every vertex renamed by one pseudo-random bijection (rows and columns alike): the
// degree distribution stays, the hot rows and columns no longer sit together at the low indices.
int64_t gen_rmat_relabel(int32_t scale, int64_t e_gen, double a, double b, double c, uint64_t seed,
                         int32_t* row_ptr, int32_t* col_idx, float* vals) {
  return gen_rmat_impl(scale, e_gen, a, b, c, seed, true, row_ptr, col_idx, vals);
}

static int64_t gen_rmat_impl(int32_t scale, int64_t e_gen, double a, double b, double c, uint64_t seed, bool relabel,
                             int32_t* row_ptr, int32_t* col_idx, float* vals) {
  std::vector<uint64_t> keys((size_t)e_gen);
  const uint32_t ta = (uint32_t)std::llround(a * 4294967296.0);
  const uint32_t tb = (uint32_t)std::llround((a + b) * 4294967296.0);
  const uint32_t tc = (uint32_t)std::llround((a + b + c) * 4294967296.0);
#pragma omp parallel for schedule(static)
  for (int64_t e = 0; e < e_gen; ++e) {
    uint32_t row = 0, col = 0;
    uint64_t h = 0;
    for (int32_t lvl = 0; lvl < scale; ++lvl) {
      if ((lvl & 1) == 0) h = rnd(seed, 200, (uint64_t)e * 32 + (uint64_t)(lvl >> 1));
      const uint32_t r = (lvl & 1) ? (uint32_t)(h >> 32) : (uint32_t)h;
      const uint32_t rb = r >= tb;                       // quadrants c, d -> lower half
      const uint32_t cb = (r >= ta && r < tb) || r >= tc;  // quadrants b, d -> right half
      row = (row << 1) | rb;
      col = (col << 1) | cb;
    }
    if (relabel) { row = relabel_vertex(row, scale, seed); col = relabel_vertex(col, scale, seed); }
    keys[(size_t)e] = ((uint64_t)row << 32) | col;
  }
#ifdef _OPENMP
  __gnu_parallel::sort(keys.begin(), keys.end());
#else
  std::sort(keys.begin(), keys.end());
#endif
  const int64_t nnz = (int64_t)(std::unique(keys.begin(), keys.end()) - keys.begin());
  const int64_t m = (int64_t)1 << scale;
  std::memset(row_ptr, 0, (size_t)(m + 1) * sizeof(int32_t));
  for (int64_t p = 0; p < nnz; ++p) {
    col_idx[p] = (int32_t)(keys[(size_t)p] & 0xFFFFFFFFull);
    row_ptr[(keys[(size_t)p] >> 32) + 1]++;
  }
  for (int64_t i = 0; i < m; ++i) row_ptr[i + 1] += row_ptr[i];
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < nnz; ++p) vals[p] = u01_open_low(rnd(seed, 1, (uint64_t)p));
  return nnz;
}

// ---------------------------------------------------------------- 3D 27-point stencil
// Grid N^3, row index (i*N + j)*N + l, diagonal `diag`, every existing neighbour in the 3x3x3 box
// gets off + sigma * N(0,1) drawn independently per stored entry; truncated at the grid boundary.
int64_t gen_stencil27_nnz(int64_t N) { const int64_t s = 3 * N - 2; return s * s * s; }
void gen_stencil27(int64_t N, float diag, float off, float sigma, uint64_t seed,
                   int32_t* row_ptr, int32_t* col_idx, float* vals) {
  const int64_t m = N * N * N;
  auto cnt = [N](int64_t t) -> int64_t { return (t > 0) + 1 + (t < N - 1); };
  int64_t p = 0;
  for (int64_t i = 0; i < N; ++i)
    for (int64_t j = 0; j < N; ++j)
      for (int64_t l = 0; l < N; ++l) {
        row_ptr[(i * N + j) * N + l] = (int32_t)p;
        p += cnt(i) * cnt(j) * cnt(l);
      }
  row_ptr[m] = (int32_t)p;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < m; ++r) {
    const int64_t l = r % N, j = (r / N) % N, i = r / (N * N);
    int64_t q = row_ptr[r];
    for (int64_t di = -1; di <= 1; ++di) {
      if (i + di < 0 || i + di >= N) continue;
      for (int64_t dj = -1; dj <= 1; ++dj) {
        if (j + dj < 0 || j + dj >= N) continue;
        for (int64_t dl = -1; dl <= 1; ++dl) {
          if (l + dl < 0 || l + dl >= N) continue;
          col_idx[q] = (int32_t)(((i + di) * N + (j + dj)) * N + (l + dl));
          if (di == 0 && dj == 0 && dl == 0) vals[q] = diag;
          else vals[q] = (float)((double)off + (double)sigma * normal01(seed, 1, (uint64_t)q));
          ++q;
        }
      }
    }
  }
}

}  // extern "C"
