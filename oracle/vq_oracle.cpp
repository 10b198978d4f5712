// vq_oracle.cpp — plain, slow, obviously-correct CPU statement of the VQ-decode linear layer.
//
// THIS IS TEST INFRASTRUCTURE.  It is the parity reference for the CUDA library and the timed
// CPU baseline of the benchmark; it is never part of the product path.  It shares no code,
// header, table or helper with the CUDA sources and includes nothing from them.
//
// What it states (GPTVQ, arXiv 2402.15319):
//   * Sec. 2.1: a codebook C_d of k centroids of dimensionality d; each group of d values of
//     the tensor is one index of ceil(log2 k) bits.
//   * Sec. 3.1: each group (block) of weights is the tuple (indices, LUT, scale factor).
//   * Sec. 3.2: indices are packed tightly; decode = look the index up; decoded values feed
//     the matrix-vector product.
//   * Sec. 4: d consecutive COLUMNS of one row form a VQ vector;
//     bits per value = log2(k)/d + k*d*b_c/l.
//   * App. A: the quantised matrix Q is constructed by looking up values of C.
// The method is a storage format, so its result has a plain definition; the oracle is that
// definition written out, every product and sum in fp64, summed left to right over k.
//
// Readings where the paper is silent (packing order, codebook order, int8 semantics) are the
// ones the library header documents; they are re-stated here in code, not shared.
//
// Parity status: every function below is pinned by tests/test_oracle_pins.py (paper-printed
// bits-per-value rows, hand-written decoded matrices, an independent big-integer bit reader,
// numpy float16 conversion, dense fp64 matmul, invariants).  Nothing here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

// IEEE binary16 -> double, exact.  Bit fields: 1 sign, 5 exponent (bias 15), 10 fraction.
double half_bits_to_double(uint16_t h) {
  const int sign = (h >> 15) & 1;
  const int expo = (h >> 10) & 0x1f;
  const int frac = h & 0x3ff;
  double v;
  if (expo == 0) {
    v = std::ldexp(static_cast<double>(frac), -24);  // subnormal: frac * 2^-24
  } else if (expo == 31) {
    v = frac ? std::nan("") : INFINITY;
  } else {
    v = std::ldexp(static_cast<double>(frac + 1024), expo - 25);  // (1024+frac) * 2^(e-15-10)
  }
  return sign ? -v : v;
}

// double -> IEEE binary16 bits, round to nearest, ties to even.
uint16_t double_to_half_bits(double x) {
  if (std::isnan(x)) return 0x7e00;
  const uint16_t sign = std::signbit(x) ? 0x8000 : 0;
  double a = std::fabs(x);
  if (a == 0.0) return sign;
  if (std::isinf(a)) return sign | 0x7c00;
  int e;  // a = m * 2^e with m in [0.5, 1)
  std::frexp(a, &e);
  int expo = e - 1;  // a = 1.f * 2^expo
  double q;          // a expressed in units of the target ulp
  if (expo < -14) {
    q = std::ldexp(a, 24);  // subnormal ulp = 2^-24
    expo = -15;
  } else {
    q = std::ldexp(a, 10 - expo);  // in [1024, 2048)
  }
  double fl = std::floor(q);
  double rem = q - fl;
  long long n = static_cast<long long>(fl);
  if (rem > 0.5 || (rem == 0.5 && (n & 1))) n += 1;
  if (expo == -15) {
    // subnormal (n < 1024) or rounded up into the smallest normal (n == 1024)
    return sign | static_cast<uint16_t>(n);
  }
  if (n == 2048) {  // mantissa overflow
    n = 1024;
    expo += 1;
  }
  if (expo > 15) return sign | 0x7c00;
  return sign | static_cast<uint16_t>(((expo + 15) << 10) | (n - 1024));
}

// Bit t of a row's little-endian bitstream = bit (t mod 8) of byte (t div 8).
inline int stream_bit(const uint8_t* row, long long t) { return (row[t / 8] >> (t % 8)) & 1; }

// Index j of a row: bits [j*b, (j+1)*b), least significant first (Sec. 2.1: one index of
// log2(k) bits per group of d values; packing order is this library's reading).
inline int read_index(const uint8_t* row, long long j, int b) {
  int v = 0;
  for (int i = 0; i < b; ++i) v |= stream_bit(row, j * b + i) << i;
  return v;
}

struct Layer {
  int N, K, d, b, Br, Bc, cb_int8;
  const uint8_t* idx;
  long long stride;
  const void* cb;
  const uint16_t* scale;
};

// Exact value of weight (n, k): Sec. 3.1 tuple + App. A look-up.  For int8 codebooks the
// value is scale * c (Sec. 2.1 symmetric quantiser x ~ s * x_int), exact in fp64.  cb_int8: 0 = fp16
// entries, 1 = int8 entries with one scale per block, 2 = int4 entries with one scale per row and
// group of 128 columns.
inline double weight_exact(const Layer& L, int n, int k) {
  const uint8_t* row = L.idx + static_cast<long long>(n) * L.stride;
  const int e = read_index(row, k / L.d, L.b);
  const long long blocks_per_row = L.K / L.Bc;
  const long long blk = static_cast<long long>(n / L.Br) * blocks_per_row + (k / L.Bc);
  const long long entries = 1LL << L.b;
  const long long at = (blk * entries + e) * L.d + (k % L.d);
  if (L.cb_int8 == 1) {
    const int8_t c = static_cast<const int8_t*>(L.cb)[at];
    return half_bits_to_double(L.scale[blk]) * static_cast<double>(c);
  }
  if (L.cb_int8 == 2) {
    // INT4 codebook with "codebook quantization groups" of 128 values (Sec. 4.2, INT4 codebooks): the
    // entry is a signed 4-bit integer (two nibbles per byte, low nibble first), the weight is that
    // integer times the scale of its row's group of 128 columns
    const uint8_t byte = static_cast<const uint8_t*>(L.cb)[at / 2];
    const int nib = (at % 2) ? (byte >> 4) : (byte & 15);
    const int c = nib >= 8 ? nib - 16 : nib;
    return half_bits_to_double(L.scale[static_cast<long long>(n) * (L.K / 128) + k / 128]) * static_cast<double>(c);
  }
  return half_bits_to_double(static_cast<const uint16_t*>(L.cb)[at]);
}

void gemm_rows(const Layer& L, const uint16_t* X, int batch, const int* rows, long long r0,
               long long r1, double* Y, double* A, long long out_rows) {
  std::vector<double> w(L.K);
  for (long long r = r0; r < r1; ++r) {
    const int n = rows ? rows[r] : static_cast<int>(r);
    for (int k = 0; k < L.K; ++k) w[k] = weight_exact(L, n, k);
    for (int m = 0; m < batch; ++m) {
      const uint16_t* x = X + static_cast<long long>(m) * L.K;
      double y = 0.0, a = 0.0;
      for (int k = 0; k < L.K; ++k) {
        const double p = w[k] * half_bits_to_double(x[k]);
        y += p;
        a += std::fabs(p);
      }
      Y[m * out_rows + r] = y;
      if (A) A[m * out_rows + r] = a;
    }
  }
}

template <class F>
void run_partitioned(long long total, int threads, F f) {
  if (threads <= 1 || total < 2) {
    f(0, total);
    return;
  }
  std::vector<std::thread> pool;
  const long long per = (total + threads - 1) / threads;
  for (int t = 0; t < threads; ++t) {
    const long long a = t * per, b = std::min(total, a + per);
    if (a >= b) break;
    pool.emplace_back([=] { f(a, b); });
  }
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// Sec. 4 "Total bits per value": log2(k)/d + k*d*b_c/l.
double ref_bpv(int k, int d, int b_c, long long l) {
  return std::log2(static_cast<double>(k)) / d + static_cast<double>(k) * d * b_c / static_cast<double>(l);
}

// Bits per value of uniform b-bit integers with one scale of s_bits per group of g (Sec. 2.1
// uniform quantiser; Sec. 5 equates g128 with 0.125 bits of overhead).
double ref_bpv_uniform(int bits, int scale_bits, int group) {
  return bits + static_cast<double>(scale_bits) / group;
}

// Bytes from one row of the index stream to the next: ceil(K/d*b/8) rounded up to 16.
long long ref_row_stride_bytes(int K, int d, int b) {
  const long long bits = static_cast<long long>(K / d) * b;
  const long long bytes = (bits + 7) / 8;
  return (bytes + 15) / 16 * 16;
}

uint16_t ref_f64_to_f16(double x) { return double_to_half_bits(x); }
double ref_f16_to_f64(uint16_t h) { return half_bits_to_double(h); }

// Pack indices I[N][K/d] (one byte each, value < 2^b) into the row bitstreams.  `idx` must be
// zero-filled or hold padding the caller wants kept: only the index bits are rewritten.
void ref_pack(int N, int K, int d, int b, const uint8_t* I, uint8_t* idx, long long stride) {
  const long long per_row = K / d;
  for (int n = 0; n < N; ++n) {
    uint8_t* row = idx + static_cast<long long>(n) * stride;
    for (long long j = 0; j < per_row; ++j) {
      const int v = I[n * per_row + j];
      for (int i = 0; i < b; ++i) {
        const long long t = j * b + i;
        const uint8_t mask = static_cast<uint8_t>(1u << (t % 8));
        if ((v >> i) & 1) row[t / 8] |= mask; else row[t / 8] &= static_cast<uint8_t>(~mask);
      }
    }
  }
}

// Sec. 3.2 step "unpack": I[n][j] = bits [j*b, (j+1)*b) of row n.
void ref_unpack(int N, int K, int d, int b, const uint8_t* idx, long long stride, uint8_t* I) {
  const long long per_row = K / d;
  for (int n = 0; n < N; ++n) {
    const uint8_t* row = idx + static_cast<long long>(n) * stride;
    for (long long j = 0; j < per_row; ++j) I[n * per_row + j] = static_cast<uint8_t>(read_index(row, j, b));
  }
}

// App. A look-up: W[n][k] = cb[blk(n,k)][I[n][k/d]][k mod d] (times the block scale for int8).
// Writes the exact fp64 values (W_exact, may be NULL) and their binary16 image (W16, may be
// NULL): a bit copy for fp16 codebooks, one round-to-nearest-even for int8*scale.
void ref_decode(int N, int K, int d, int b, int Br, int Bc, int cb_int8, const uint8_t* idx,
                long long stride, const void* cb, const uint16_t* scale, double* W_exact,
                uint16_t* W16) {
  const Layer L{N, K, d, b, Br, Bc, cb_int8, idx, stride, cb, scale};
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) {
      const double w = weight_exact(L, n, k);
      const long long at = static_cast<long long>(n) * K + k;
      if (W_exact) W_exact[at] = w;
      if (W16) W16[at] = double_to_half_bits(w);
    }
}

// Sec. 3.2 mat-vec on decoded values: Y[m][r] = sum_k W[n_r][k] * X[m][k], fp64, k ascending.
// rows == NULL: all N rows (out_rows = N).  Otherwise only the listed rows, Y is [batch][n_sel].
// A (may be NULL) receives sum_k |W*X|, the scale of the acceptance tolerance.
void ref_gemm(int N, int K, int d, int b, int Br, int Bc, int cb_int8, const uint8_t* idx,
              long long stride, const void* cb, const uint16_t* scale, const uint16_t* X, int batch,
              const int* rows, long long n_sel, double* Y, double* A, int threads) {
  const Layer L{N, K, d, b, Br, Bc, cb_int8, idx, stride, cb, scale};
  const long long total = rows ? n_sel : N;
  run_partitioned(total, threads, [&](long long a, long long e) { gemm_rows(L, X, batch, rows, a, e, Y, A, total); });
}

// Textbook dense product on an fp64 matrix, same summation order (k ascending).
void ref_dense_gemm(int N, int K, const double* W, const uint16_t* X, int batch, double* Y) {
  for (int m = 0; m < batch; ++m)
    for (int n = 0; n < N; ++n) {
      double y = 0.0;
      for (int k = 0; k < K; ++k) y += W[static_cast<long long>(n) * K + k] * half_bits_to_double(X[static_cast<long long>(m) * K + k]);
      Y[static_cast<long long>(m) * N + n] = y;
    }
}

// Uniform INT4 group-128 yard-stick (Sec. 2.1 x ~ s*x_int; Sec. 5 INT4 g128):
// w[n][k] = scale[n][k/128] * (q[n][k] - 8), q = nibble (k mod 2) of byte k/2, low nibble first.
void ref_int4g128_gemm(int N, int K, const uint8_t* q, const uint16_t* scale, const uint16_t* X,
                       int batch, double* Y, double* A, int threads) {
  run_partitioned(N, threads, [&](long long a, long long e) {
    std::vector<double> w(K);
    for (long long n = a; n < e; ++n) {
      for (int k = 0; k < K; ++k) {
        const uint8_t byte = q[n * (K / 2) + k / 2];
        const int nib = (k % 2) ? (byte >> 4) : (byte & 15);
        w[k] = half_bits_to_double(scale[n * (K / 128) + k / 128]) * static_cast<double>(nib - 8);
      }
      for (int m = 0; m < batch; ++m) {
        double y = 0.0, s = 0.0;
        for (int k = 0; k < K; ++k) {
          const double p = w[k] * half_bits_to_double(X[static_cast<long long>(m) * K + k]);
          y += p;
          s += std::fabs(p);
        }
        Y[static_cast<long long>(m) * N + n] = y;
        if (A) A[static_cast<long long>(m) * N + n] = s;
      }
    }
  });
}

int ref_hardware_threads() { return static_cast<int>(std::thread::hardware_concurrency()); }

}  // extern "C"
