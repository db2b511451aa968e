// Host-side constants of the method: the 2M modulus set of Section 4, the roots s_j (Section 2), the byte
// weights of the residue kernels and the CRT weights (Section 3.1), computed with a small multi-limb integer.
#include "common.cuh"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

namespace gemm2m {

// Greedy coprime set of 2M moduli in [1, 256], descending (Section 4), followed by the first non-2M moduli of the same
// greedy walk that are coprime to all of them (hybrid 2M/3M, Sections 3 and 4).
static const int kModuli[kMaxMod] = {241, 233, 229, 221, 205, 197, 193, 181, 173, 157, 149, 137, 113,
                                     109, 101, 97,  89,  73,  61,  53,  37,  29,  256, 253, 251, 249};

// The set available to the real Ozaki-II scheme (Section 4): the same greedy walk without the 2M condition.
static const int kRealModuli[kMaxReal] = {256, 255, 253, 251, 247, 241, 239, 233, 229, 227,
                                          223, 217, 211, 199, 197, 193, 191, 181, 179, 173};

// The analogous set for the Eisenstein integers (Sections 3.2 and 4): coprime products of primes congruent to 1 mod 3.
static const int kEisModuli[kMaxEis] = {247, 241, 229, 223, 217, 211, 199, 193, 181, 163, 157, 151,
                                        139, 127, 109, 103, 97,  79,  73,  67,  61,  43,  37};

int modulus_value(int j) { return kModuli[j]; }
int eis_modulus_value(int j) { return kEisModuli[j]; }

int eis_cube_root(int j) {   // smallest s > 1 with s^2 + s + 1 = 0 (mod m)
    const int m = kEisModuli[j];
    for (int s = 2; s < m; ++s)
        if ((s * s + s + 1) % m == 0) return s;
    return 0;
}
// d = 2s + 1 = s - s^2 is a square root of -3: in the coordinates (u + v sqrt(-3))/2 of the Eisenstein integers the two ring
// homomorphisms are u +- d v (up to the unit 2), which is Eq. (2a) with d in the place of s.
static int eis_sqrt_minus3(int j) { return (2 * eis_cube_root(j) + 1) % kEisModuli[j]; }
int real_modulus_value(int j) { return kRealModuli[j]; }

int modulus_root(int j) {   // smallest positive s with s^2 = -1 (mod m); 0 for a non-2M modulus
    if (j >= kMax2M) return 0;
    const int m = kModuli[j];
    for (int s = 1; s < m; ++s)
        if ((s * s + 1) % m == 0) return s;
    return 0;
}

static inline int sym_mod(int64_t x, int m) {   // representative in [-(m-1)/2, (m-1)/2]; even m: [-m/2, m/2 - 1]
    int r = (int)(x % m);
    if (r < 0) r += m;
    if (r > (m - 1) / 2) r -= m;
    return r;
}

static int inv_mod(int a, int m) {   // a^-1 mod m by search (m <= 256)
    a %= m;
    if (a < 0) a += m;
    for (int x = 1; x < m; ++x)
        if ((a * x) % m == 1) return x;
    return 0;
}

// ---- non-negative multi-limb integer, base 2^32, little endian ----
struct Big {
    std::vector<uint32_t> w;
    void trim() { while (!w.empty() && w.back() == 0) w.pop_back(); }
    static Big from(uint64_t v) { Big b; b.w = {(uint32_t)v, (uint32_t)(v >> 32)}; b.trim(); return b; }
    void mul_small(uint32_t f) {
        uint64_t carry = 0;
        for (auto& limb : w) { uint64_t t = (uint64_t)limb * f + carry; limb = (uint32_t)t; carry = t >> 32; }
        if (carry) w.push_back((uint32_t)carry);
        trim();
    }
    uint32_t divmod_small(uint32_t d) {   // in-place quotient, returns remainder
        uint64_t rem = 0;
        for (size_t i = w.size(); i-- > 0;) { uint64_t t = (rem << 32) | w[i]; w[i] = (uint32_t)(t / d); rem = t % d; }
        trim();
        return (uint32_t)rem;
    }
    uint32_t mod_small(uint32_t d) const { Big c = *this; return c.divmod_small(d); }
    int bit_length() const {
        if (w.empty()) return 0;
        int top = 32 - __builtin_clz(w.back());
        return (int)(w.size() - 1) * 32 + top;
    }
    uint64_t bits(int pos, int count) const {   // count <= 64 bits starting at bit pos
        uint64_t out = 0;
        for (int b = 0; b < count; ++b) {
            int p = pos + b;
            size_t limb = (size_t)(p >> 5);
            if (limb < w.size() && ((w[limb] >> (p & 31)) & 1u)) out |= (1ull << b);
        }
        return out;
    }
    void shr(int bits) {   // 0 < bits < 32
        uint32_t c = 0;
        for (size_t i = w.size(); i-- > 0;) { const uint32_t n = w[i] << (32 - bits); w[i] = (w[i] >> bits) | c; c = n; }
        trim();
    }
    void add_small(uint32_t v) {
        uint64_t carry = v;
        for (auto& limb : w) { if (!carry) break; const uint64_t t = (uint64_t)limb + carry; limb = (uint32_t)t; carry = t >> 32; }
        if (carry) w.push_back((uint32_t)carry);
    }
    void add(const Big& o) {
        if (w.size() < o.w.size()) w.resize(o.w.size(), 0u);
        uint64_t carry = 0;
        for (size_t i = 0; i < w.size(); ++i) { const uint64_t t = (uint64_t)w[i] + (i < o.w.size() ? o.w[i] : 0u) + carry; w[i] = (uint32_t)t; carry = t >> 32; }
        if (carry) w.push_back((uint32_t)carry);
    }
    void sub(const Big& o) {   // *this >= o
        int64_t borrow = 0;
        for (size_t i = 0; i < w.size(); ++i) {
            int64_t t = (int64_t)w[i] - (i < o.w.size() ? (int64_t)o.w[i] : 0) - borrow;
            borrow = t < 0;
            if (t < 0) t += 4294967296LL;
            w[i] = (uint32_t)t;
        }
        trim();
    }
    void sub_one() { for (auto& limb : w) { if (limb-- != 0) break; } trim(); }
    void shr1() { uint32_t c = 0; for (size_t i = w.size(); i-- > 0;) { uint32_t n = w[i] & 1u; w[i] = (w[i] >> 1) | (c << 31); c = n; } trim(); }
    double to_double() const { double v = 0; for (size_t i = w.size(); i-- > 0;) v = v * 4294967296.0 + w[i]; return v; }
};

static Big product_of(int nmod, const int* mods = kModuli) {
    Big M = Big::from(1);
    for (int j = 0; j < nmod; ++j) M.mul_small((uint32_t)mods[j]);
    return M;
}

// mods: the modulus list; n2: how many of the first nmod are 2M moduli (the others take the plain weights for both parts).
// The tables are functions of the modulus count alone: each is built once per process and copied out afterwards, so that a
// call's host cost is its launches, not multi-word arithmetic.
template <class T, int N, class F>
static void memoised(int nmod, T* out, F&& build) {
    static T cache[N + 1];
    static std::once_flag once[N + 1];
    std::call_once(once[nmod], [&] { build(&cache[nmod]); });
    *out = cache[nmod];
}

static void build_residue_table_for(const int* mods, int nmod, int n2, ResidueTable* t, int (*root)(int) = modulus_root) {
    std::memset(t, 0, sizeof(*t));
    t->nmod = nmod;
    t->n2 = n2;
    for (int j = 0; j < nmod; ++j) {
        const int m = mods[j], s = j < n2 ? root(j) : 1;
        t->m[j] = m;
        t->s[j] = s;
        t->inv_m[j] = 1.0f / (float)m;
        int64_t p = 1;   // 256^b mod m
        uint32_t w[12], ws[12];
        for (int b = 0; b < 12; ++b) {
            w[b] = (uint32_t)(uint8_t)(int8_t)sym_mod(p, m);
            ws[b] = (uint32_t)(uint8_t)(int8_t)sym_mod(p * s, m);
            p = (p * 256) % m;
        }
        // Reduction constants.  x = (dp4a sum of the real part) +- (dp4a sum of the imaginary part) is bounded by xmax below
        // (digits: four unsigned bytes, then up to eight balanced ones).  The real chain starts at the bit pattern of
        // Y0 = the first multiple of 256 m that is >= 2^23 + xmax, so the integer sum is the float y = Y0 + x exactly
        // (2^23 <= y < 2^24, one unit per ulp).  With cq = 1.5 2^23 - Y0/m (an integer), the exact value of
        // fma(y, inv_m, cq) is 1.5 2^23 + x/m + y d, d = inv_m - 1/m, which rounds to 1.5 2^23 + rint(x/m) because
        // |y d| < 1/(2m), the least distance of x/m from a rounding boundary (residue_reduction_margin checks it).
        // Y0 is a multiple of 256 and so is the bit pattern of 1.5 2^23: the low byte of y - (1.5 2^23 + q) m is that of x - q m.
        int64_t xmax = 0;
        for (int b = 0; b < 12; ++b) {
            const int64_t digit = b < 4 ? 255 : 128;
            xmax += digit * (std::abs((int)(int8_t)w[b]) + std::abs((int)(int8_t)ws[b]));
        }
        const int64_t step = 256LL * m;
        const int64_t y0 = (((1LL << 23) + xmax + step - 1) / step) * step;
        t->magic[j] = (int32_t)(0x4B000000LL + (y0 - (1LL << 23)));
        t->cq[j] = (float)(12582912LL - y0 / m);
        t->xmax[j] = (int32_t)xmax;
        auto pack = [](const uint32_t* v) { return v[0] | (v[1] << 8) | (v[2] << 16) | (v[3] << 24); };
        t->w_lo[j] = pack(w);
        t->w_hi[j] = pack(w + 4);
        t->w_top[j] = pack(w + 8);
        t->ws_lo[j] = pack(ws);
        t->ws_hi[j] = pack(ws + 4);
        t->ws_top[j] = pack(ws + 8);
    }
}

void build_residue_table(int nmod, ResidueTable* t) {
    memoised<ResidueTable, kMaxMod>(nmod, t, [&](ResidueTable* c) { build_residue_table_for(kModuli, nmod, count_2m(nmod), c); });
}
void build_residue_table_eis(int nmod, ResidueTable* t) {
    memoised<ResidueTable, kMaxEis>(nmod, t, [&](ResidueTable* c) { build_residue_table_for(kEisModuli, nmod, nmod, c, eis_sqrt_minus3); });
}
void build_residue_table_real(int nmod, ResidueTable* t) {
    memoised<ResidueTable, kMaxReal>(nmod, t, [&](ResidueTable* c) { build_residue_table_for(kRealModuli, nmod, 0, c); });
}

// 2^e / (2 (Y0 + xmax) |n m - 2^e|) for inv_m = n 2^-e: the factor by which the error term of the residue kernels'
// quotient estimate stays below the distance 1/(2m) of x/m from the nearest rounding boundary (must exceed 1).
double residue_reduction_margin(const ResidueTable& t, int j) {
    int ex = 0;
    const float mant = std::frexp(t.inv_m[j], &ex);          // inv_m = mant 2^ex, 0.5 <= mant < 1
    const int64_t n = (int64_t)std::ldexp((double)mant, 24); // exact: 24-bit significand
    const int e = 24 - ex;
    const int64_t y0 = (int64_t)(t.magic[j] - 0x4B000000) + (1LL << 23);
    const int64_t dev = std::llabs(n * t.m[j] - (1LL << e));
    if (dev == 0) return 1e30;
    return (double)(1LL << e) / (2.0 * (double)(y0 + t.xmax[j]) * (double)dev);
}

// Epilogue constants of one batch entry: the reduction constants of the residue kernels for this modulus (the bound used
// there, twelve digits of both parts, covers four unsigned bytes, the 2^31 correction and one stored residue).
static void fill_mod_entry(ModTable* t, int p, const int* mods, int j) {
    ResidueTable r;
    build_residue_table_for(mods, j + 1, 0, &r);
    t->m[p] = r.m[j];
    t->inv_m[p] = r.inv_m[j];
    t->w[p] = r.w_lo[j];
    // the epilogue contracts the bytes of x + 2^31: take 2^31 mod m out again
    t->y0[p] = r.magic[j] - sym_mod(1LL << 31, r.m[j]);
    t->cq[p] = r.cq[j];
}

static void build_mod_table_for(int nmod, bool per_plane, ModTable* t) {
    std::memset(t, 0, sizeof(*t));
    const int n2 = count_2m(nmod);
    int p = 0;
    auto put = [&](int j) { fill_mod_entry(t, p, kModuli, j); ++p; };
    if (!per_plane) {
        for (int j = 0; j < nmod; ++j) put(j);
    } else {
        for (int rep = 0; rep < 2; ++rep)
            for (int j = 0; j < n2; ++j) put(j);
        for (int rep = 0; rep < 3; ++rep)
            for (int j = n2; j < nmod; ++j) put(j);
    }
    t->nplanes = p;
}

void build_mod_table(int nmod, bool per_plane, ModTable* t) {
    if (per_plane) memoised<ModTable, kMaxMod>(nmod, t, [&](ModTable* c) { build_mod_table_for(nmod, true, c); });
    else memoised<ModTable, kMaxMod>(nmod, t, [&](ModTable* c) { build_mod_table_for(nmod, false, c); });
}

void build_mod_table_eis(int nmod, ModTable* t) {   // one entry per plane: the + planes, then the - planes
    memoised<ModTable, kMaxEis>(nmod, t, [&](ModTable* c) {
        std::memset(c, 0, sizeof(*c));
        for (int p = 0; p < 2 * nmod; ++p) fill_mod_entry(c, p, kEisModuli, p % nmod);
        c->nplanes = 2 * nmod;
    });
}

void build_mod_table_real(int nmod, ModTable* t) {
    memoised<ModTable, kMaxReal>(nmod, t, [&](ModTable* c) {
        std::memset(c, 0, sizeof(*c));
        for (int j = 0; j < nmod; ++j) fill_mod_entry(c, j, kRealModuli, j);
        c->nplanes = nmod;
    });
}

// Folded CRT weights: g_j = sym(2^-1 q_j mod m_j), h_j = sym(s_j 2^-1 q_j mod m_j), q_j = (M/m_j)^-1 mod m_j.
static void folded_weights(int nmod, int j, const Big& M, Big* W, int* g, int* h, const int* mods = kModuli, int n2 = kMax2M) {
    const int m = mods[j];
    *W = M;
    W->divmod_small((uint32_t)m);
    const int q = inv_mod((int)W->mod_small((uint32_t)m), m);
    if (mods == kEisModuli) {
        // The residue planes hold u +- d v = 2 (a + s b), 2 (a + s^2 b), so the products are 4 C+, 4 C-.  With
        // C = (U + V sqrt(-3))/2:  U = C+ + C- = 4^-1 (sum of the planes), V = (C+ - C-)/d = -(4d)^-1 (minus plane - plus plane).
        const int quarter = inv_mod(4, m);
        *g = sym_mod((int64_t)quarter * q, m);
        *h = sym_mod(-(int64_t)inv_mod(4 * eis_sqrt_minus3(j) % m, m) * q, m);
        return;
    }
    if (j >= n2) {                  // 3M modulus (Eq. (1)) or real scheme (Section 3.1): no factor besides q_j
        *g = *h = sym_mod(q, m);
        return;
    }
    const int half = (m + 1) / 2;   // 2^-1 mod m (Section 2)
    *g = sym_mod((int64_t)half * q, m);
    *h = sym_mod((int64_t)modulus_root(j) * half % m * q, m);
    (void)nmod;
}

static void build_crt_table_for(const int* mods, int nmod, int n2, CrtTable* t) {
    std::memset(t, 0, sizeof(*t));
    t->nmod = nmod;
    t->n2 = n2;
    const Big M = product_of(nmod, mods);
    Big half = M;   // (M-1)/2 bounds every |G_j|
    half.sub_one();
    half.shr1();
    t->nchunks = (half.bit_length() + kChunkBits - 1) / kChunkBits;
    if (t->nchunks < 1) t->nchunks = 1;
    // digits of M; the top digit in use takes every remaining bit (M may be one bit longer than (M-1)/2: 41 bits there)
    for (int c = 0; c < t->nchunks; ++c)
        t->Mc[c] = (double)M.bits(c * kChunkBits, c + 1 < t->nchunks ? kChunkBits : 60);
    for (int j = 0; j < nmod; ++j) {
        Big W;
        int g, h;
        folded_weights(nmod, j, M, &W, &g, &h, mods, mods == kModuli ? kMax2M : mods == kEisModuli ? kMaxEis : 0);
        Big Gr = W, Gi = W;
        Gr.mul_small((uint32_t)std::abs(g));
        Gi.mul_small((uint32_t)std::abs(h));
        for (int c = 0; c < kMaxChunks; ++c) {
            t->gr[j][c] = (g < 0 ? -1.0 : 1.0) * (double)Gr.bits(c * kChunkBits, kChunkBits);
            t->gi[j][c] = (h < 0 ? -1.0 : 1.0) * (double)Gi.bits(c * kChunkBits, kChunkBits);
        }
    }
    t->q_hi = std::ldexp(1.0, kChunkBits * (t->nchunks - 1)) / M.to_double();
    t->q_lo = t->nchunks > 1 ? std::ldexp(t->q_hi, -kChunkBits) : 0.0;
}

void build_crt_table(int nmod, CrtTable* t) {
    memoised<CrtTable, kMaxMod>(nmod, t, [&](CrtTable* c) { build_crt_table_for(kModuli, nmod, count_2m(nmod), c); });
}
void build_crt_table_eis(int nmod, CrtTable* t) {
    memoised<CrtTable, kMaxEis>(nmod, t, [&](CrtTable* c) {
        build_crt_table_for(kEisModuli, nmod, nmod, c);
        // result = (U + V sqrt(-3))/2: the real part is U/2, the imaginary part V sqrt(3)/2 with the factor as a double-double
        c->re_shift = -1;
        c->im_hi = 0x1.bb67ae8584caap-1;
        c->im_lo = 0x1.cec95d0b5c1e3p-55;
    });
}
void build_crt_table_real(int nmod, CrtTable* t) {
    memoised<CrtTable, kMaxReal>(nmod, t, [&](CrtTable* c) { build_crt_table_for(kRealModuli, nmod, 0, c); });
}

// herk: the plane order of the rank-k family (see build_post_mma_table_herk).
static void build_post_mma_table_for(const int* mods, int nmod, int n2, PostMmaTable* t, bool herk = false) {
    std::memset(t, 0, sizeof(*t));
    const int n3 = nmod - n2, herk_half = 16 * ((n2 + 15) / 16);
    const int planes = herk ? 2 * herk_half : 2 * n2 + 3 * n3;
    auto slot = [&](int plane) { return herk && plane >= n2 ? herk_half + (plane - n2) : plane; };
    const Big M = product_of(nmod, mods);
    const int ndig = (M.bit_length() + 7) / 8;                        // bytes of a residue modulo M
    if (ndig > 4 * kPostMaxNB) std::abort();                          // cannot happen: M < 2^185
    Big ksum[2];                                                      // sum over the planes of the weights, per part
    auto put = [&](int part, int plane, const Big& W, int coef) {    // weight of `plane` in `part` = coef W (mod M), as bytes
        if (coef == 0) return;
        Big G = W;
        G.mul_small((uint32_t)std::abs(coef));                        // below M/2: |coef| <= m_j / 2
        if (coef < 0) { Big R = M; R.sub(G); G = R; }
        ksum[part].add(G);
        for (int p = 0; p < ndig; ++p) t->digit[part][slot(plane)][p] = (uint8_t)G.bits(8 * p, 8);
    };
    for (int j = 0; j < nmod; ++j) {
        Big W;
        int g, h;
        folded_weights(nmod, j, M, &W, &g, &h, mods, n2);
        if (j < n2) {                      // Eq. (2c): X_r takes (C- + C+) g, X_i takes (C- - C+) h
            put(0, j, W, g);
            put(0, n2 + j, W, g);
            put(1, j, W, -h);
            put(1, n2 + j, W, h);
        } else {                           // Eq. (1): X_r takes (P1 - P2) g, X_i takes (P3 - P1 - P2) g
            const int j3 = j - n2, p1 = 2 * n2 + j3, p2 = p1 + n3, p3 = p2 + n3;
            put(0, p1, W, g);
            put(0, p2, W, -g);
            put(1, p1, W, -g);
            put(1, p2, W, -g);
            put(1, p3, W, g);
        }
    }
    PostConsts& c = t->c;
    t->nmod = nmod;
    c.planes = planes;
    c.ks = (planes + 31) / 32;
    c.nb = 2 * ((ndig + 7) / 8);           // 32-bit chunks (4 digits each), an even number of them: a lane of the kernel holds whole chunks
    // M in base 2^32: balanced lower digits, the top digit takes what remains; each stored times its power of 2^32
    Big rest = M;
    for (int k = 0; k < c.nb; ++k) {
        double d;
        if (k + 1 < c.nb) {
            const uint32_t low = rest.w.empty() ? 0u : rest.w[0];
            if (!rest.w.empty()) { rest.w.erase(rest.w.begin()); rest.trim(); }
            d = (double)low;
            if (low >= 0x80000000u) { d -= 4294967296.0; rest.add_small(1); }
        } else {
            d = rest.to_double();          // below 2^53: exact
        }
        c.Mc[k] = std::ldexp(d, 32 * k);
    }
    // The kernel contracts (residue + 128) with the weights: 128 times the sum of a part's weights comes off again, chunk
    // by chunk, together with the offset 1.5 2^52 of the integer-to-double conversion (top chunk: all remaining bits, < 2^46).
    for (int part = 0; part < 2; ++part) {
        Big K = ksum[part];
        K.mul_small(128);
        for (int k = 0; k < c.nb; ++k) {
            const double d = k + 1 < c.nb ? (double)K.bits(32 * k, 32) : (double)K.bits(32 * k, 52);
            c.off[part][k] = std::ldexp(6755399441055744.0 + d, 32 * k);
        }
    }
    c.inv_M = 1.0 / M.to_double();
    for (int s = 0; s < c.ks; ++s)
        for (int q = 0; q < c.nb; ++q)
            for (int hh = 0; hh < 2; ++hh)
                for (int lane = 0; lane < 32; ++lane) {
                    const int g = lane >> 2, tt = lane & 3;
                    // B-operand column g of block q is accumulator column (lane tC = g / 2, register b = g % 2); lanes 0, 1 of
                    // a quad collect the real part, lanes 2, 3 the imaginary part, each lane nb pairs of neighbouring digits
                    const int tc = g >> 1, b = g & 1, part = tc >> 1, p = 2 * ((tc & 1) * c.nb + q) + b;
                    uint32_t word = 0;
                    for (int r = 0; r < 4; ++r) {
                        // K index 4 tt + r of the half: the complex GEMMs' kernel loads its operand with the planes in their order,
                        // the rank-k kernel gathers the planes tt, tt + 4, tt + 8, tt + 12 into one register
                        const int plane = 32 * s + 16 * hh + (herk ? tt + 4 * r : 4 * tt + r);
                        const uint32_t byte = plane < planes ? (uint32_t)t->digit[part][plane][p] : 0u;
                        word |= byte << (8 * r);
                    }
                    t->bfrag[((s * c.nb + q) * 2 + hh) * 32 + lane] = word;
                }
}

void build_post_mma_table(int nmod, PostMmaTable* t) {
    memoised<PostMmaTable, kMaxMod>(nmod, t, [&](PostMmaTable* c) { build_post_mma_table_for(kModuli, nmod, count_2m(nmod), c); });
}
void build_post_mma_table_herk(int nmod, PostMmaTable* t) {
    static PostMmaTable cache[kMax2M + 1];
    static std::once_flag once[kMax2M + 1];
    std::call_once(once[nmod], [&] { build_post_mma_table_for(kModuli, nmod, nmod, &cache[nmod], true); });
    *t = cache[nmod];
}
void build_post_mma_table_eis(int nmod, PostMmaTable* t) {
    memoised<PostMmaTable, kMaxEis>(nmod, t, [&](PostMmaTable* c) {
        build_post_mma_table_for(kEisModuli, nmod, nmod, c);
        c->c.re_shift = -1;                      // result = (U + V sqrt(-3))/2, the factor sqrt(3)/2 as a double-double
        c->c.im_hi = 0x1.bb67ae8584caap-1;
        c->c.im_lo = 0x1.cec95d0b5c1e3p-55;
    });
}

static void build_crt_table_int_for(int nmod, CrtTableInt* t) {
    std::memset(t, 0, sizeof(*t));
    t->nmod = nmod;
    const Big M = product_of(nmod);
    t->M = (int64_t)M.bits(0, 63);
    for (int j = 0; j < nmod; ++j) {
        Big W;
        int g, h;
        folded_weights(nmod, j, M, &W, &g, &h);
        t->W[j] = (int64_t)W.bits(0, 63);
        t->gr[j] = g;
        t->gi[j] = h;
        t->m[j] = kModuli[j];
    }
}

void build_crt_table_int(int nmod, CrtTableInt* t) {
    memoised<CrtTableInt, kMaxMod>(nmod, t, [&](CrtTableInt* c) { build_crt_table_int_for(nmod, c); });
}

// floor(log2((M-1)/2)) for the first nmod moduli of a list.
static int budget_bits(int nmod, const int* mods) {
    Big half = product_of(nmod, mods);
    half.sub_one();
    half.shr1();
    return half.bit_length() - 1;
}

// Scaling budget: P_t = floor(log2((M-1)/2)) split between rows of A and columns of B; c_k = ceil(log2(2k)/2).
ScaleTargets scale_targets(int nmod, int64_t k, bool herk) {
    ScaleTargets s;
    memoised<int, kMaxMod>(nmod, &s.Pt, [&](int* c) { *c = budget_bits(nmod, kModuli); });
    s.PA = (s.Pt + 1) / 2;
    s.PB = s.Pt / 2;
    if (herk) s.PA = s.PB = s.Pt / 2;
    s.ck = 0;
    const int64_t kk = k > 0 ? k : 1;
    while ((1ull << (2 * s.ck)) < (uint64_t)(2 * kk)) ++s.ck;
    return s;
}

// Eisenstein variant: lattice rounding moves a point by up to 0.578 and the coordinates U, V of an entry c of the product are
// bounded by 2|c|: c_k = ceil(log2(5k)/2) keeps them below 2^P_t as long as the scaled parts reach 4 (P_B - c_k >= 2).
ScaleTargets scale_targets_eis(int nmod, int64_t k) {
    ScaleTargets s;
    memoised<int, kMaxEis>(nmod, &s.Pt, [&](int* c) { *c = budget_bits(nmod, kEisModuli); });
    s.PA = (s.Pt + 1) / 2;
    s.PB = s.Pt / 2;
    s.ck = 0;
    const int64_t kk = k > 0 ? k : 1;
    while ((1ull << (2 * s.ck)) < (uint64_t)(5 * kk)) ++s.ck;
    return s;
}

// Real scheme (Section 3.1): a row has k real terms, c_k = ceil(log2(k)/2).
ScaleTargets scale_targets_real(int nmod, int64_t k) {
    ScaleTargets s;
    memoised<int, kMaxReal>(nmod, &s.Pt, [&](int* c) { *c = budget_bits(nmod, kRealModuli); });
    s.PA = (s.Pt + 1) / 2;
    s.PB = s.Pt / 2;
    s.ck = 0;
    const int64_t kk = k > 0 ? k : 1;
    while ((1ull << (2 * s.ck)) < (uint64_t)kk) ++s.ck;
    return s;
}

// The accumulators must stay inside int32 (the epilogue works on x + 2^31 as an unsigned 32-bit number).
static constexpr int64_t kAccLimit = 0x7FFFFFFFLL;

int64_t gemm_k_limit_real() { return kAccLimit / (128 * 128); }   // the modulus 256 comes first

int64_t gemm_k_limit_eis() { const int64_t h = (kEisModuli[0] - 1) / 2; return kAccLimit / (h * h); }

int64_t gemm_k_limit(int nmod) {
    // largest |residue|: 120 for the 2M moduli (241 comes first), 128 once the hybrid adds the modulus 256
    const int64_t h = nmod > kMax2M ? 128 : (kModuli[0] - 1) / 2;
    return kAccLimit / (h * h);
}

}  // namespace gemm2m
