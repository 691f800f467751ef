// Host-side constants of the method: modulus selection (Section 5.1), Eq. 3 capacity,
// CRT weights (Section 5.2), and the small per-modulus reduction constants.
// Multiword integers are little-endian arrays of 32-bit words.
#include <math.h>
#include <string.h>

#include <mutex>

#include "ozk_common.cuh"

namespace ozk {
namespace {

constexpr int kW = 8;  // host big integers: 256 bits
struct Big {
  uint32_t w[kW];
};

Big big_from(uint64_t v) {
  Big b;
  memset(&b, 0, sizeof b);
  b.w[0] = (uint32_t)v;
  b.w[1] = (uint32_t)(v >> 32);
  return b;
}
Big big_mul_small(const Big& a, uint32_t m) {
  Big r;
  uint64_t carry = 0;
  for (int i = 0; i < kW; ++i) {
    uint64_t t = (uint64_t)a.w[i] * m + carry;
    r.w[i] = (uint32_t)t;
    carry = t >> 32;
  }
  return r;
}
Big big_div_small(const Big& a, uint32_t m, uint32_t* rem) {
  Big q;
  uint64_t r = 0;
  for (int i = kW - 1; i >= 0; --i) {
    uint64_t t = (r << 32) | a.w[i];
    q.w[i] = (uint32_t)(t / m);
    r = t % m;
  }
  if (rem) *rem = (uint32_t)r;
  return q;
}
Big big_add(const Big& a, const Big& b) {
  Big r;
  uint64_t carry = 0;
  for (int i = 0; i < kW; ++i) {
    uint64_t t = (uint64_t)a.w[i] + b.w[i] + carry;
    r.w[i] = (uint32_t)t;
    carry = t >> 32;
  }
  return r;
}
int big_cmp(const Big& a, const Big& b) {
  for (int i = kW - 1; i >= 0; --i)
    if (a.w[i] != b.w[i]) return a.w[i] < b.w[i] ? -1 : 1;
  return 0;
}
Big big_shl(const Big& a, int s) {
  Big r;
  memset(&r, 0, sizeof r);
  int ws = s / 32, bs = s % 32;
  for (int i = kW - 1; i >= ws; --i) {
    uint64_t v = (uint64_t)a.w[i - ws] << bs;
    if (bs && i - ws - 1 >= 0) v |= a.w[i - ws - 1] >> (32 - bs);
    r.w[i] = (uint32_t)v;
  }
  return r;
}
int big_bits(const Big& a) {
  for (int i = kW - 1; i >= 0; --i)
    if (a.w[i]) return 32 * i + 32 - __builtin_clz(a.w[i]);
  return 0;
}
double big_to_double(const Big& a) {
  double r = 0.0;
  for (int i = kW - 1; i >= 0; --i) r = r * 4294967296.0 + (double)a.w[i];
  return r;
}

// The doubled E2M1 magnitudes (Section 3).
const int kS[15] = {0, 1, 2, 3, 4, 6, 8, 12, -1, -2, -3, -4, -6, -8, -12};

// Section 5.1: every residue class of m holds some c0 + 13 c1.
bool two_limb_representable(int m) {
  bool seen[512];
  for (int i = 0; i < m; ++i) seen[i] = false;
  int count = 0;
  for (int i = 0; i < 15; ++i)
    for (int j = 0; j < 15; ++j) {
      int v = ((kS[i] + 13 * kS[j]) % m + m) % m;
      if (!seen[v]) {
        seen[v] = true;
        ++count;
      }
    }
  return count == m;
}
int gcd_int(int a, int b) {
  while (b) {
    int t = a % b;
    a = b;
    b = t;
  }
  return a;
}
Big product_of(const int* m, int L) {
  Big P = big_from(1);
  for (int i = 0; i < L; ++i) P = big_mul_small(P, (uint32_t)m[i]);
  return P;
}

// Section 5.1: 169 first, then descending, pairwise coprime, no other multiple of 13.  The search is
// run once per process; later calls copy a prefix of its result.
struct ModulusList {
  int m[kMaxModuli];
  int n;
};
const ModulusList& modulus_list() {
  static const ModulusList list = [] {
    ModulusList r;
    r.n = 0;
    for (int m = 169; m >= 2 && r.n < kMaxModuli; --m) {
      if (m != 169 && m % 13 == 0) continue;
      if (!two_limb_representable(m)) continue;
      bool ok = true;
      for (int i = 0; i < r.n; ++i) ok = ok && gcd_int(m, r.m[i]) == 1;
      if (ok) r.m[r.n++] = m;
    }
    return r;
  }();
  return list;
}

}  // namespace

int host_select_moduli(int count, int* out) {
  const ModulusList& list = modulus_list();
  const int n = count < list.n ? count : list.n;
  for (int i = 0; i < n; ++i) out[i] = list.m[i];
  return n;
}

// Eq. 3 for a c-bit integer width: 2 K 2^(2c) < P, capped at max_bits (53 in Section 4.2; up to 62 in
// the extended-capacity mode).
int host_capacity_bits(int64_t K, int L, int max_bits) {
  int m[kMaxModuli];
  if (L < 1 || L > kMaxModuli || host_select_moduli(L, m) != L) return -1;
  Big P = product_of(m, L);
  Big twoK = big_from(2 * (uint64_t)(K < 1 ? 1 : K));
  int c = 0;
  while (c < max_bits) {
    if (big_bits(twoK) + 2 * (c + 1) >= 32 * kW) break;
    if (big_cmp(big_shl(twoK, 2 * (c + 1)), P) >= 0) break;
    ++c;
  }
  return c;
}

namespace {
bool build_modulus_table(int L, ModulusTable* t);
bool build_crt_table(int L, CrtTable* t);
}  // namespace

// The per-L tables are built once per process and copied out afterwards.
bool host_build_modulus_table(int L, ModulusTable* t) {
  if (L < 1 || L > kMaxModuli) return false;
  static std::mutex mu;
  static bool have[kMaxModuli + 1];
  static ModulusTable cache[kMaxModuli + 1];
  std::lock_guard<std::mutex> lock(mu);
  if (!have[L]) {
    if (!build_modulus_table(L, &cache[L])) return false;
    have[L] = true;
  }
  *t = cache[L];
  return true;
}

bool host_build_crt_table(int L, CrtTable* t) {
  if (L < 1 || L > kMaxModuli) {
    memset(t, 0, sizeof *t);
    return false;
  }
  static std::mutex mu;
  static bool have[kMaxModuli + 1];
  static CrtTable cache[kMaxModuli + 1];
  std::lock_guard<std::mutex> lock(mu);
  if (!have[L]) {
    if (!build_crt_table(L, &cache[L])) {
      *t = cache[L];
      return false;
    }
    have[L] = true;
  }
  *t = cache[L];
  return true;
}

namespace {

bool build_modulus_table(int L, ModulusTable* t) {
  if (L < 1 || L > kMaxModuli || host_select_moduli(L, t->m) != L) return false;
  t->L = L;
  for (int i = 0; i < L; ++i) {
    uint32_t m = (uint32_t)t->m[i];
    t->recip[i] = (uint32_t)(0x100000000ull / m);
    for (int p = 0; p < 8; ++p) {
      unsigned long long pw = 1;  // 2^(8 p) mod m
      for (int k = 0; k < 8 * p; ++k) pw = pw * 2 % m;
      t->c8[i][p] = (uint8_t)pw;
    }
    unsigned long long off = 1;  // 2^62 mod m
    for (int k = 0; k < 62; ++k) off = off * 2 % m;
    t->off62[i] = (int)off;
  }
  for (int i = L; i < kMaxModuli; ++i) {
    t->m[i] = 1, t->recip[i] = 0, t->off62[i] = 0;
    for (int p = 0; p < 8; ++p) t->c8[i][p] = 0;
  }
  return true;
}

// Section 5.2: w_l = M_l (M_l^-1 mod m_l), M_l = P / m_l; S = sum r_l w_l <= sum (m_l - 1) w_l.
bool build_crt_table(int L, CrtTable* t) {
  memset(t, 0, sizeof *t);
  if (L < 1 || L > kMaxModuli || host_select_moduli(L, t->m) != L) return false;
  t->L = L;
  Big P = product_of(t->m, L);
  Big smax = big_from(0);
  for (int l = 0; l < L; ++l) {
    uint32_t m = (uint32_t)t->m[l], rem = 0;
    Big Ml = big_div_small(P, m, &rem);
    if (rem != 0) return false;
    uint32_t Mmod = 0;
    big_div_small(Ml, m, &Mmod);
    uint32_t inv = 0;
    for (uint32_t x = 1; x < m; ++x)
      if ((uint64_t)Mmod * x % m == 1) inv = x;
    if (m == 1) inv = 0;
    Big w = big_mul_small(Ml, inv);
    for (int i = 0; i < kCrtWords; ++i) t->w[l][i] = w.w[i];
    for (int i = kCrtWords; i < kW; ++i)
      if (w.w[i]) return false;
    smax = big_add(smax, big_mul_small(w, m - 1));
  }
  if (big_bits(smax) > 32 * kCrtWords) return false;
  t->words = (big_bits(smax) + 31) / 32;
  if (t->words < 2) t->words = 2;
  for (int i = 0; i < kCrtWords; ++i) t->P[i] = P.w[i];
  Big h = big_div_small(P, 2, nullptr);
  for (int i = 0; i < kCrtWords; ++i) t->halfP[i] = h.w[i];
  {
    const int nw = big_bits(P) <= 128 ? 4 : 5;  // 2^(32 nw) - P
    uint64_t borrow = 0;
    for (int i = 0; i < 5; ++i) {
      const uint64_t d = (uint64_t)0 - P.w[i] - borrow;
      t->negP[i] = i < nw ? (uint32_t)d : 0u;
      borrow = (d >> 32) & 1u;
    }
  }
  t->inv_P = 1.0 / big_to_double(P);
  t->p_bits = big_bits(P);
  t->q_mul = 0, t->q_word = 0, t->q_bit = 0;
  if (t->p_bits >= 85 && t->p_bits <= 160) {
    // largest c with c P 2^28 <= 2^(52 + shift) (2^28 - 1), by bisection
    const int shift = t->p_bits - 21;
    const Big rhs = big_shl(big_from((1ull << 28) - 1), 52 + shift);
    uint64_t lo = 0, hi = 0xFFFFFFFFull;
    while (lo < hi) {
      const uint64_t mid = (lo + hi + 1) / 2;
      if (big_cmp(big_shl(big_mul_small(P, (uint32_t)mid), 28), rhs) <= 0) lo = mid; else hi = mid - 1;
    }
    t->q_mul = (uint32_t)lo;
    t->q_word = shift / 32;
    t->q_bit = shift % 32;
  }
  for (int tile = 0; tile < 3; ++tile)
    for (int lane = 0; lane < 32; ++lane) {
      const int col = lane >> 2, q = lane & 3;
      const int digit = tile < 2 ? 4 * (col / 2) + 2 * tile + col % 2 : 16 + col;
      for (int reg = 0; reg < 2; ++reg) {
        uint32_t v = 0;
        for (int n = 0; n < 4; ++n) {
          const int l = q + 16 * reg + 4 * n;
          if (l < L && digit < 4 * kCrtWords) v |= ((t->w[l][digit / 4] >> (8 * (digit % 4))) & 0xFFu) << (8 * n);
        }
        t->bfrag[tile][lane][reg] = v;
      }
    }
  return true;
}

}  // namespace

}  // namespace ozk
