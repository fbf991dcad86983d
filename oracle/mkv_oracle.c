/*
 * mkv_oracle.c -- plain, slow CPU oracle for mixed-format (FP8 + TQ3) paged decode attention.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may include, link or call this file;
 * it shares no code, header, table or constant generator with the CUDA library.  It exists so
 * that tests can compare the CUDA path with an implementation that can be checked against the
 * paper by eye.
 *
 * What it follows:
 *   - Section 3.1 (tiers): Recent/Anchor pages are FP8, Stale pages are TQ3, "a three-bit
 *     rotated scalar quantizer", "norm-corrected packed layout".
 *   - Section 4.1: per stale page and KV head TQ3 stores three-bit rotated key codes, an FP16
 *     key-norm correction, three-bit value codes and FP16 scale/zero metadata.
 *   - Section 4 ("Evaluated profiles", last paragraph): FP8-to-TQ3 conversion is a
 *     normalize-rotate-pack operation.
 *   - Section 3.3, Eq. (softmax-merge): attention over the concatenated logical cache, and the
 *     per-partition (m_j, l_j, O_j) merge that is algebraically equal to it.
 *   - Eq. (kv-per-token), Eq. (effective-bits), Section 6.3 byte counters: byte accounting.
 *
 * The paper fixes the structure of TQ3 but not its constants; the readings used here (rotation =
 * randomised Walsh-Hadamard, Lloyd-Max N(0,1) codebook rounded to fp16, norm correction
 * g = |x|/|c|, per-channel asymmetric 3-bit values, fp32 encoder with a fixed operation order)
 * are stated where they are used below.  Parity status per function:
 *   pinned by the paper / mathematics / a library: e4m3 codec, fp16 conversion, byte accounting,
 *     codebook values (Lloyd-Max), key round trip and norm preservation, value round-trip
 *     bounds, attention (dense special case, brute force, partition invariance, indexing).
 *   pinned by the paper's byte counters (Section 6.3): the sizes of pages of 16 M tokens, i.e. one
 *     value scale/zero pair per channel and PAGE.
 *   parity unpinned (fixed only by the readings made here): choice of rotation, definition of
 *     the norm correction, value quantiser being un-rotated, tie-breaking, FP8 scale handling,
 *     bit positions of the packed records, order of tiles and metadata inside a page of 16 M tokens.
 *
 * Floating point: the encoder works in fp32, one IEEE round-to-nearest operation at a time
 * (compile with -ffp-contract=off, no fast-math).  Dequantisation and attention work in fp64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_T 16 /* tokens per page, and per tile of a page of 16 M tokens */
#define ORC_MAXD 256

/* ------------------------------------------------------------------------------------------
 * scalar formats
 * ---------------------------------------------------------------------------------------- */

float orc_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* OCP e4m3fn: 1 sign, 4 exponent (bias 7), 3 mantissa; no infinity; 0x7F / 0xFF are NaN;
 * subnormals step 2^-9; largest finite value 448. */
double orc_e4m3_decode(uint8_t b)
{
    int s = b >> 7, e = (b >> 3) & 15, m = b & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    v = (e == 0) ? ldexp((double)m / 8.0, -6) : ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* fp32 -> e4m3fn, round to nearest even, saturate to +-448.  Written as a nearest-value
 * search over the 127 finite non-negative codes so that it can be checked by eye. */
uint8_t orc_e4m3_encode(float x)
{
    uint8_t sign = (uint8_t)(signbit(x) ? 0x80 : 0x00);
    double a = fabs((double)x), best_err = 0.0;
    int best = 0, c;
    if (isnan(x)) return (uint8_t)(sign | 0x7F);
    if (a >= 448.0) return (uint8_t)(sign | 0x7E);
    for (c = 0; c <= 0x7E; ++c) {
        double err = fabs(orc_e4m3_decode((uint8_t)c) - a);
        if (c == 0 || err < best_err || (err == best_err && (c & 1) == 0)) {
            best = c;
            best_err = err;
        }
    }
    return (uint8_t)(sign | best);
}

/* fp32 -> fp16 bits, round to nearest even, saturating at +-65504 (never produces inf). */
uint16_t orc_f32_to_f16_sat(float x)
{
    _Float16 h;
    uint16_t u;
    if (x > 65504.0f) x = 65504.0f;
    if (x < -65504.0f) x = -65504.0f;
    h = (_Float16)x;
    memcpy(&u, &h, 2);
    return u;
}

float orc_f16_to_f32(uint16_t u)
{
    _Float16 h;
    memcpy(&h, &u, 2);
    return (float)h;
}

/* ------------------------------------------------------------------------------------------
 * TQ3 codebook (Section 3.1: three-bit scalar quantizer of the rotated, normalised key)
 * Record format 1: 8-level Lloyd-Max quantiser of N(0,1): magnitudes = nearest fp16 to the optimal
 *   levels, thresholds = midpoints of adjacent magnitudes (exact in fp32).
 * Record format 2: the same quantiser with every magnitude moved to the nearest number that the 8-bit
 *   float e4m3 holds exactly (three mantissa bits): 0.25, 0.75, 1.375, 2.25; thresholds = midpoints
 *   0.5, 1.0625, 1.8125.  A reader can then feed the codes to FP8 arithmetic without any rounding.
 *   The paper prints no codebook; this one costs about 1 % more Gaussian distortion than format 1
 *   (pinned in the tests against a Lloyd iteration).  Everything else of the encoder is unchanged.
 * The format is a property of a pool; the functions below follow the one selected here.
 * ---------------------------------------------------------------------------------------- */
static const float ORC_C1[4] = {0.2451171875f, 0.755859375f, 1.34375f, 2.15234375f};
static const float ORC_B1[3] = {0.50048828125f, 1.0498046875f, 1.748046875f};
static const float ORC_C2[4] = {0.25f, 0.75f, 1.375f, 2.25f};
static const float ORC_B2[3] = {0.5f, 1.0625f, 1.8125f};
static int orc_format = 1;
#define ORC_C (orc_format == 2 ? ORC_C2 : ORC_C1)
#define ORC_B (orc_format == 2 ? ORC_B2 : ORC_B1)

/* select the record format (1 or 2) used by every function of this file; not to be changed while
 * a call is running on another thread */
int orc_set_format(int f)
{
    if (f != 1 && f != 2) return -1;
    orc_format = f;
    return 0;
}
int orc_get_format(void) { return orc_format; }

float orc_codebook_level(int j) { return ORC_C[j & 3]; }
float orc_codebook_threshold(int j) { return ORC_B[j % 3]; }

/* ------------------------------------------------------------------------------------------
 * TQ3 key encoder: normalize - rotate - quantise - norm-correct, one token vector x[0..d).
 *   sigma[i] in {+1,-1}: the random signs of the randomised Hadamard rotation R = d^-1/2 H diag(sigma)
 *   code[i]  = mag | sign<<2   (mag 0..3 indexes ORC_C, sign 1 = negative)
 *   g        = fp16(|x| / |c|) : the FP16 key-norm correction
 * Every arithmetic step is a single fp32 operation, in the order written.
 * ---------------------------------------------------------------------------------------- */
void orc_tq3_encode_key(const float* x, int d, const int8_t* sigma, uint8_t* code, uint16_t* g)
{
    float a[ORC_MAXD], e[ORC_MAXD], t[ORC_MAXD];
    float n2, nx, nc2, nc, t1, t2, t3;
    int i, h;

    /* 1. sign flip (exact) */
    for (i = 0; i < d; ++i) a[i] = (sigma[i] < 0) ? -x[i] : x[i];
    /* 2. unnormalised Walsh-Hadamard transform, Sylvester order, strides ascending */
    for (h = 1; h < d; h <<= 1)
        for (i = 0; i < d; ++i)
            if ((i & h) == 0) {
                float u = a[i], v = a[i + h];
                a[i] = u + v;
                a[i + h] = u - v;
            }
    /* 3. |x|^2 by a butterfly all-reduce, strides ascending; |x| */
    for (i = 0; i < d; ++i) e[i] = x[i] * x[i];
    for (h = 1; h < d; h <<= 1) {
        for (i = 0; i < d; ++i) t[i] = e[i] + e[i ^ h];
        memcpy(e, t, sizeof(float) * (size_t)d);
    }
    n2 = e[0];
    nx = sqrtf(n2);
    /* 4. a[i]/nx has unit mean square; compare |a[i]| with threshold * nx (strict >) */
    t1 = ORC_B[0] * nx;
    t2 = ORC_B[1] * nx;
    t3 = ORC_B[2] * nx;
    for (i = 0; i < d; ++i) {
        float w = fabsf(a[i]);
        int mag = (w > t1) + (w > t2) + (w > t3);
        int sgn = (a[i] < 0.0f) ? 1 : 0; /* +-0 -> positive */
        code[i] = (uint8_t)(mag | (sgn << 2));
    }
    /* 5. |c|^2 with the same butterfly; g = |x| / |c| */
    for (i = 0; i < d; ++i) e[i] = ORC_C[code[i] & 3] * ORC_C[code[i] & 3];
    for (h = 1; h < d; h <<= 1) {
        for (i = 0; i < d; ++i) t[i] = e[i] + e[i ^ h];
        memcpy(e, t, sizeof(float) * (size_t)d);
    }
    nc2 = e[0];
    nc = sqrtf(nc2);
    *g = (nx == 0.0f) ? (uint16_t)0 : orc_f32_to_f16_sat(nx / nc);
}

/* TQ3 key decoder in fp64: k^ = g * d^-1/2 * sigma .* (H c)   (the inverse rotation is applied
 * to the key; the rotated-query shortcut is deliberately not used here). */
void orc_tq3_decode_key(const uint8_t* code, uint16_t g, int d, const int8_t* sigma, double* out)
{
    double y[ORC_MAXD];
    double gg = (double)orc_f16_to_f32(g), rs = 1.0 / sqrt((double)d);
    int i, h;
    for (i = 0; i < d; ++i) {
        double c = (double)ORC_C[code[i] & 3];
        y[i] = (code[i] & 4) ? -c : c;
    }
    for (h = 1; h < d; h <<= 1)
        for (i = 0; i < d; ++i)
            if ((i & h) == 0) {
                double u = y[i], v = y[i + h];
                y[i] = u + v;
                y[i + h] = u - v;
            }
    for (i = 0; i < d; ++i) out[i] = gg * rs * (sigma[i] < 0 ? -y[i] : y[i]);
}

/* TQ3 value encoder for one full page of T tokens: v[t*d + c], t < T.  Asymmetric uniform 3-bit
 * quantiser per channel over ALL tokens of the page; scale and zero stored as fp16 (Section 4.1:
 * "three-bit value codes, and FP16 scale/zero" per Stale page and KV head). */
void orc_tq3_encode_value_block(const float* v, int d, int T, uint8_t* code /*[T*d] token-major*/,
                                uint16_t* sc /*[d]*/, uint16_t* zp /*[d]*/)
{
    int c, t;
    for (c = 0; c < d; ++c) {
        float mn = v[c], mx = v[c], scf, zpf;
        for (t = 1; t < T; ++t) {
            float u = v[(int64_t)t * d + c];
            if (u < mn) mn = u;
            if (u > mx) mx = u;
        }
        sc[c] = orc_f32_to_f16_sat((mx - mn) / 7.0f);
        zp[c] = orc_f32_to_f16_sat(mn);
        scf = orc_f16_to_f32(sc[c]);
        zpf = orc_f16_to_f32(zp[c]);
        for (t = 0; t < T; ++t) {
            int q = 0;
            if (scf != 0.0f) {
                float r = rintf((v[(int64_t)t * d + c] - zpf) / scf); /* half to even */
                if (r < 0.0f) r = 0.0f;
                if (r > 7.0f) r = 7.0f;
                q = (int)r;
            }
            code[(int64_t)t * d + c] = (uint8_t)q;
        }
    }
}

/* the 16-token page */
void orc_tq3_encode_value_page(const float* v, int d, uint8_t* code /*[16*d] token-major*/,
                               uint16_t* sc /*[d]*/, uint16_t* zp /*[d]*/)
{
    orc_tq3_encode_value_block(v, d, ORC_T, code, sc, zp);
}

double orc_tq3_decode_value(uint8_t code, uint16_t sc, uint16_t zp)
{
    return (double)orc_f16_to_f32(sc) * (double)code + (double)orc_f16_to_f32(zp);
}

/* ------------------------------------------------------------------------------------------
 * Packed records (Section 4.1: a Stale page's codes, scales and metadata sit in one record per page).
 * The values (codes, g, scale, zero) are the semantics; the positions below are a wire choice
 * that the paper does not print.  All sections start on 16-byte boundaries.
 *
 * FP8 record of (page, kv head), 32*d bytes:
 *    [0, 16d)    K  e4m3  [token t][dim i]          (token-major)
 *    [16d, 32d)  V  e4m3  [channel c][token t]      (channel-major)
 *
 * TQ3 record of (page, kv head), 16*d + 32 bytes, NB = d/16 blocks of 16:
 *    [0, 6d)          K codes   32 "lanes" x (3*NB/4) 32-bit words
 *    [6d, 12d)        V codes   32 "lanes" x (3*NB/4) 32-bit words
 *    [12d, 12d+32)    g[16]     fp16, token order
 *    [12d+32, 16d+32) V scale/zero fp16, [NB/2 block pairs][8 rows][8 halves]
 * A lane's words are stored in chunks of four (16 bytes): word w of lane L sits at
 * (w/4)*512 + L*16 + (w%4)*4; when only two words remain (d = 128: words 4,5) that last chunk
 * is 8 bytes per lane: 512 + L*8 + (w-4)*4.
 *
 * Format 1.  K code of token t, rotated dim i:  block kb = i/16, slot s = i%16.
 *    lane = 4*(t%8) + (s%8)/2 ; register r = (t/8) + 2*(s/8) ; half = s%2
 *    word triple j = kb/4 (words 3j, 3j+1, 3j+2 = A, B, C), nibble n = 2*r + half
 *    kb%4 == 0: A bits [4n,4n+2] = code        kb%4 == 1: B bits [4n,4n+2] = code
 *    kb%4 == 2: C bits [4n,4n+1] = mag, A bit 4n+3 = sign
 *    kb%4 == 3: C bits [4n+2,4n+3] = mag, B bit 4n+3 = sign
 * Format 2 re-cuts the K section only (same words per lane, same triples A, B, C):
 *    K code of token t, rotated dim i:  step s = i/32, k = i%32.
 *    lane = 4*(t%8) + (k%16)/4 ; triple j = s/2 ; e = 4*(s%2) + 2*(t/8) + k/16 ; nibble n = 4*(e%2) + k%4
 *    e = 0,1: A bits [4n,4n+2] = code          e = 2,3: B bits [4n,4n+2] = code
 *    e = 4,5: C bits [4n,4n+1] = mag, A bit 4n+3 = sign
 *    e = 6,7: C bits [4n+2,4n+3] = mag, B bit 4n+3 = sign
 *    (four consecutive dims of one token are the four nibbles of one half-word: a reader turns them
 *    into four 8-bit operands with one byte-table lookup)
 * V code of token t, channel c (both formats):  block cb = c/16, row = c%16.
 *    lane = 4*(row%8) + (t%8)/2 ; register r = (row/8) + 2*(t/8) ; half = t%2
 *    word triple j = cb/4; group = (cb%4)/2; field k = 4*(cb%2) + r; stream bit = 3k + bit
 *    each (group, half) is a 24-bit stream of three bytes S0 S1 S2:
 *      group 0: half 0 -> W0.b0, W0.b1, W1.b0   half 1 -> W0.b2, W0.b3, W1.b2
 *      group 1: half 0 -> W1.b1, W2.b0, W2.b1   half 1 -> W1.b3, W2.b2, W2.b3
 * V scale/zero of channel c = 16*cb + row: half index (cb/2)*64 + (row%8)*8 + 4*(cb%2)
 *    + 2*is_zero + (row/8).
 * ---------------------------------------------------------------------------------------- */

int64_t orc_fp8_record_bytes(int d) { return 32 * (int64_t)d; }
int64_t orc_tq3_record_bytes(int d) { return 16 * (int64_t)d + 32; }

static int64_t lane_word_offset(int d, int lane, int w)
{
    int words = 3 * (d / 16) / 4; /* per lane: 6 (d=128) or 12 (d=256) */
    int chunk = w / 4, rem = words - 4 * chunk;
    if (rem >= 4) return (int64_t)chunk * 512 + lane * 16 + (w % 4) * 4;
    return (int64_t)chunk * 512 + lane * 8 + (w % 4) * 4; /* trailing 2-word chunk */
}

static void set_bit(uint8_t* rec, int64_t byte_off, int bit, int val)
{
    int64_t b = byte_off + (bit >> 3);
    if (val)
        rec[b] = (uint8_t)(rec[b] | (1u << (bit & 7)));
    else
        rec[b] = (uint8_t)(rec[b] & ~(1u << (bit & 7)));
}

static int get_bit(const uint8_t* rec, int64_t byte_off, int bit)
{
    return (rec[byte_off + (bit >> 3)] >> (bit & 7)) & 1;
}

/* position of bit `bit` (0,1 = magnitude, 2 = sign) of the K code (t, i): byte offset of the
 * 32-bit word inside the record and the bit index inside that word */
static void kcode_pos(int d, int t, int i, int bit, int64_t* word_off, int* wbit)
{
    if (orc_format == 2) {
        int s = i / 32, k = i % 32;
        int lane = 4 * (t % 8) + (k % 16) / 4, j = s / 2, e = 4 * (s % 2) + 2 * (t / 8) + k / 16;
        int n = 4 * (e % 2) + k % 4, w;
        if (e < 2)      { w = 3 * j;     *wbit = 4 * n + bit; }
        else if (e < 4) { w = 3 * j + 1; *wbit = 4 * n + bit; }
        else if (e < 6) {
            if (bit < 2) { w = 3 * j + 2; *wbit = 4 * n + bit; }
            else         { w = 3 * j;     *wbit = 4 * n + 3; }
        } else {
            if (bit < 2) { w = 3 * j + 2; *wbit = 4 * n + 2 + bit; }
            else         { w = 3 * j + 1; *wbit = 4 * n + 3; }
        }
        *word_off = lane_word_offset(d, lane, w);
        return;
    }
    int kb = i / 16, s = i % 16;
    int lane = 4 * (t % 8) + (s % 8) / 2, r = (t / 8) + 2 * (s / 8), half = s % 2;
    int j = kb / 4, n = 2 * r + half, w;
    switch (kb % 4) {
    case 0: w = 3 * j;     *wbit = 4 * n + bit; break;
    case 1: w = 3 * j + 1; *wbit = 4 * n + bit; break;
    case 2:
        if (bit < 2) { w = 3 * j + 2; *wbit = 4 * n + bit; }
        else         { w = 3 * j;     *wbit = 4 * n + 3; }
        break;
    default:
        if (bit < 2) { w = 3 * j + 2; *wbit = 4 * n + 2 + bit; }
        else         { w = 3 * j + 1; *wbit = 4 * n + 3; }
        break;
    }
    *word_off = lane_word_offset(d, lane, w);
}

static void vcode_pos(int d, int t, int c, int bit, int64_t* word_off, int* wbit)
{
    static const int W[2][2][3] = {{{0, 0, 1}, {0, 0, 1}}, {{1, 2, 2}, {1, 2, 2}}};   /* word */
    static const int Y[2][2][3] = {{{0, 1, 0}, {2, 3, 2}}, {{1, 0, 1}, {3, 2, 3}}};   /* byte */
    int cb = c / 16, row = c % 16;
    int lane = 4 * (row % 8) + (t % 8) / 2, r = (row / 8) + 2 * (t / 8), half = t % 2;
    int j = cb / 4, grp = (cb % 4) / 2, k = 4 * (cb % 2) + r, sb = 3 * k + bit;
    int w = 3 * j + W[grp][half][sb / 8];
    *wbit = 8 * Y[grp][half][sb / 8] + (sb % 8);
    *word_off = 6 * (int64_t)d + lane_word_offset(d, lane, w);
}

static int64_t vmeta_half_index(int c, int is_zero)
{
    int cb = c / 16, row = c % 16;
    return (int64_t)(cb / 2) * 64 + (row % 8) * 8 + 4 * (cb % 2) + 2 * is_zero + (row / 8);
}

void orc_tq3_pack_record(int d, const uint8_t* kcode /*[16][d]*/, const uint16_t* g /*[16]*/,
                         const uint8_t* vcode /*[16][d]*/, const uint16_t* sc, const uint16_t* zp,
                         uint8_t* rec)
{
    int t, i, bit, wbit;
    int64_t off;
    memset(rec, 0, (size_t)orc_tq3_record_bytes(d));
    for (t = 0; t < ORC_T; ++t)
        for (i = 0; i < d; ++i)
            for (bit = 0; bit < 3; ++bit) {
                kcode_pos(d, t, i, bit, &off, &wbit);
                set_bit(rec, off, wbit, (kcode[t * d + i] >> bit) & 1);
                vcode_pos(d, t, i, bit, &off, &wbit);
                set_bit(rec, off, wbit, (vcode[t * d + i] >> bit) & 1);
            }
    for (t = 0; t < ORC_T; ++t) memcpy(rec + 12 * (int64_t)d + 2 * t, &g[t], 2);
    for (i = 0; i < d; ++i) {
        memcpy(rec + 12 * (int64_t)d + 32 + 2 * vmeta_half_index(i, 0), &sc[i], 2);
        memcpy(rec + 12 * (int64_t)d + 32 + 2 * vmeta_half_index(i, 1), &zp[i], 2);
    }
}

void orc_tq3_unpack_record(int d, const uint8_t* rec, uint8_t* kcode, uint16_t* g, uint8_t* vcode,
                           uint16_t* sc, uint16_t* zp)
{
    int t, i, bit, wbit;
    int64_t off;
    for (t = 0; t < ORC_T; ++t)
        for (i = 0; i < d; ++i) {
            int kc = 0, vc = 0;
            for (bit = 0; bit < 3; ++bit) {
                kcode_pos(d, t, i, bit, &off, &wbit);
                kc |= get_bit(rec, off, wbit) << bit;
                vcode_pos(d, t, i, bit, &off, &wbit);
                vc |= get_bit(rec, off, wbit) << bit;
            }
            kcode[t * d + i] = (uint8_t)kc;
            vcode[t * d + i] = (uint8_t)vc;
        }
    for (t = 0; t < ORC_T; ++t) memcpy(&g[t], rec + 12 * (int64_t)d + 2 * t, 2);
    for (i = 0; i < d; ++i) {
        memcpy(&sc[i], rec + 12 * (int64_t)d + 32 + 2 * vmeta_half_index(i, 0), 2);
        memcpy(&zp[i], rec + 12 * (int64_t)d + 32 + 2 * vmeta_half_index(i, 1), 2);
    }
}

/* FP8 record from fp32 K,V of one page and head (k[t*d+i], v[t*d+c]); tokens >= n_valid are
 * written as zero bytes.  stored = e4m3(x * (1/scale)), 1/scale rounded once to fp32. */
void orc_fp8_pack_record(int d, const float* k, const float* v, int n_valid, float k_scale,
                         float v_scale, uint8_t* rec)
{
    float ik = 1.0f / k_scale, iv = 1.0f / v_scale;
    int t, i;
    memset(rec, 0, (size_t)orc_fp8_record_bytes(d));
    for (t = 0; t < n_valid; ++t)
        for (i = 0; i < d; ++i) {
            rec[t * d + i] = orc_e4m3_encode(k[t * d + i] * ik);
            rec[16 * d + i * ORC_T + t] = orc_e4m3_encode(v[t * d + i] * iv);
        }
}

/* exact fp32 dequantisation of an FP8 record (the input of the FP8 -> TQ3 demotion) */
void orc_fp8_unpack_record_f32(int d, const uint8_t* rec, float k_scale, float v_scale, float* k,
                               float* v)
{
    int t, i;
    for (t = 0; t < ORC_T; ++t)
        for (i = 0; i < d; ++i) {
            k[t * d + i] = (float)orc_e4m3_decode(rec[t * d + i]) * k_scale;
            v[t * d + i] = (float)orc_e4m3_decode(rec[16 * d + i * ORC_T + t]) * v_scale;
        }
}

/* Retier(p, TQ3) of Algorithm 1, data part: FP8 record -> TQ3 record of one (page, head). */
void orc_demote_record(int d, const uint8_t* fp8_rec, float k_scale, float v_scale,
                       const int8_t* sigma, uint8_t* tq3_rec)
{
    float* k = (float*)malloc(sizeof(float) * ORC_T * (size_t)d);
    float* v = (float*)malloc(sizeof(float) * ORC_T * (size_t)d);
    uint8_t* kc = (uint8_t*)malloc(ORC_T * (size_t)d);
    uint8_t* vc = (uint8_t*)malloc(ORC_T * (size_t)d);
    uint16_t g[ORC_T], sc[ORC_MAXD], zp[ORC_MAXD];
    int t;
    orc_fp8_unpack_record_f32(d, fp8_rec, k_scale, v_scale, k, v);
    for (t = 0; t < ORC_T; ++t) orc_tq3_encode_key(k + t * d, d, sigma, kc + t * d, &g[t]);
    orc_tq3_encode_value_page(v, d, vc, sc, zp);
    orc_tq3_pack_record(d, kc, g, vc, sc, zp, tq3_rec);
    free(k); free(v); free(kc); free(vc);
}

/* TQ3 record straight from fp32 K,V of a full page (used when the harness encodes Stale pages
 * from the bf16 originals). */
void orc_tq3_record_from_f32(int d, const float* k, const float* v, const int8_t* sigma,
                             uint8_t* tq3_rec)
{
    uint8_t* kc = (uint8_t*)malloc(ORC_T * (size_t)d);
    uint8_t* vc = (uint8_t*)malloc(ORC_T * (size_t)d);
    uint16_t g[ORC_T], sc[ORC_MAXD], zp[ORC_MAXD];
    int t;
    for (t = 0; t < ORC_T; ++t) orc_tq3_encode_key(k + t * d, d, sigma, kc + t * d, &g[t]);
    orc_tq3_encode_value_page(v, d, vc, sc, zp);
    orc_tq3_pack_record(d, kc, g, vc, sc, zp, tq3_rec);
    free(kc); free(vc);
}

/* ------------------------------------------------------------------------------------------
 * Pages of T = 16 M tokens (Section 4.1: the measured prototype stores blocks of 1,792 tokens,
 * the fast-arithmetic one blocks of 832; Section 5.4 counts their physical bytes).  A page is M
 * tiles of 16 tokens.  Keys are coded per token, so a key tile is the key part of the 16-token
 * record; value scale and zero are per channel over ALL T tokens of the page (one scale/zero
 * pair per channel and page, which is what amortises the value metadata to ~3.04 bit/scalar).
 *
 *   FP8 page of (page, kv head), M * 32 d bytes: tile m = the 16-token FP8 record of tokens
 *       [16 m, 16 m + 16) at offset m * 32 d.
 *   TQ3 page of (page, kv head), M * (12 d + 32) + 4 d bytes: tile m at offset m * (12 d + 32)
 *       = [key codes 6 d | value codes 6 d | g[16] 32 B] of its 16 tokens, laid out as in the
 *       16-token record; then the page's value scale/zero (4 d bytes, same order as there).
 *   M = 1 gives exactly the 16-token records.
 * ---------------------------------------------------------------------------------------- */
int64_t orc_fp8_block_bytes(int d, int M) { return (int64_t)M * orc_fp8_record_bytes(d); }
int64_t orc_tq3_tile_bytes(int d) { return 12 * (int64_t)d + 32; }
int64_t orc_tq3_block_bytes(int d, int M) { return M * orc_tq3_tile_bytes(d) + 4 * (int64_t)d; }

void orc_tq3_pack_block(int d, int M, const uint8_t* kcode /*[16M][d]*/, const uint16_t* g /*[16M]*/,
                        const uint8_t* vcode /*[16M][d]*/, const uint16_t* sc, const uint16_t* zp, uint8_t* rec)
{
    uint8_t* tmp = (uint8_t*)malloc((size_t)orc_tq3_record_bytes(d));
    int64_t tile = orc_tq3_tile_bytes(d);
    int m;
    for (m = 0; m < M; ++m) {
        orc_tq3_pack_record(d, kcode + (int64_t)m * ORC_T * d, g + m * ORC_T, vcode + (int64_t)m * ORC_T * d, sc, zp, tmp);
        memcpy(rec + m * tile, tmp, (size_t)tile);
    }
    memcpy(rec + M * tile, tmp + tile, (size_t)(4 * d));     /* scale/zero: the same in every tile's record */
    free(tmp);
}

void orc_tq3_unpack_block(int d, int M, const uint8_t* rec, uint8_t* kcode, uint16_t* g, uint8_t* vcode,
                          uint16_t* sc, uint16_t* zp)
{
    uint8_t* tmp = (uint8_t*)malloc((size_t)orc_tq3_record_bytes(d));
    int64_t tile = orc_tq3_tile_bytes(d);
    int m;
    for (m = 0; m < M; ++m) {
        memcpy(tmp, rec + m * tile, (size_t)tile);
        memcpy(tmp + tile, rec + M * tile, (size_t)(4 * d));
        orc_tq3_unpack_record(d, tmp, kcode + (int64_t)m * ORC_T * d, g + m * ORC_T, vcode + (int64_t)m * ORC_T * d, sc, zp);
    }
    free(tmp);
}

/* TQ3 page straight from fp32 K,V of a full page of 16 M tokens (k[t*d+i], v[t*d+c]) */
void orc_tq3_block_from_f32(int d, int M, const float* k, const float* v, const int8_t* sigma, uint8_t* rec)
{
    int T = ORC_T * M, t;
    uint8_t* kc = (uint8_t*)malloc((size_t)T * d);
    uint8_t* vc = (uint8_t*)malloc((size_t)T * d);
    uint16_t* g = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)T);
    uint16_t sc[ORC_MAXD], zp[ORC_MAXD];
    for (t = 0; t < T; ++t) orc_tq3_encode_key(k + (int64_t)t * d, d, sigma, kc + (int64_t)t * d, &g[t]);
    orc_tq3_encode_value_block(v, d, T, vc, sc, zp);
    orc_tq3_pack_block(d, M, kc, g, vc, sc, zp, rec);
    free(kc); free(vc); free(g);
}

void orc_fp8_pack_block(int d, int M, const float* k, const float* v, int n_valid, float k_scale, float v_scale,
                        uint8_t* rec)
{
    int m;
    for (m = 0; m < M; ++m) {
        int n = n_valid - m * ORC_T;
        n = n < 0 ? 0 : (n > ORC_T ? ORC_T : n);
        orc_fp8_pack_record(d, k + (int64_t)m * ORC_T * d, v + (int64_t)m * ORC_T * d, n, k_scale, v_scale,
                            rec + m * orc_fp8_record_bytes(d));
    }
}

void orc_fp8_unpack_block_f32(int d, int M, const uint8_t* rec, float k_scale, float v_scale, float* k, float* v)
{
    int m;
    for (m = 0; m < M; ++m)
        orc_fp8_unpack_record_f32(d, rec + m * orc_fp8_record_bytes(d), k_scale, v_scale, k + (int64_t)m * ORC_T * d,
                                  v + (int64_t)m * ORC_T * d);
}

/* Retier(p, TQ3), data part, for a page of 16 M tokens */
void orc_demote_block(int d, int M, const uint8_t* fp8_block, float k_scale, float v_scale, const int8_t* sigma,
                      uint8_t* tq3_block)
{
    int T = ORC_T * M;
    float* k = (float*)malloc(sizeof(float) * (size_t)T * d);
    float* v = (float*)malloc(sizeof(float) * (size_t)T * d);
    orc_fp8_unpack_block_f32(d, M, fp8_block, k_scale, v_scale, k, v);
    orc_tq3_block_from_f32(d, M, k, v, sigma, tq3_block);
    free(k); free(v);
}

void orc_promote_record(int d, const uint8_t* tq3_rec, float k_scale, float v_scale, const int8_t* sigma,
                        uint8_t* fp8_rec);

/* Promote(p), data part, for a page of 16 M tokens: every tile is rebuilt like a 16-token record
 * whose scale/zero are the page's */
void orc_promote_block(int d, int M, const uint8_t* tq3_block, float k_scale, float v_scale, const int8_t* sigma,
                       uint8_t* fp8_block)
{
    uint8_t* tmp = (uint8_t*)malloc((size_t)orc_tq3_record_bytes(d));
    int64_t tile = orc_tq3_tile_bytes(d);
    int m;
    for (m = 0; m < M; ++m) {
        memcpy(tmp, tq3_block + m * tile, (size_t)tile);
        memcpy(tmp + tile, tq3_block + M * tile, (size_t)(4 * d));
        orc_promote_record(d, tmp, k_scale, v_scale, sigma, fp8_block + m * orc_fp8_record_bytes(d));
    }
    free(tmp);
}

/* ------------------------------------------------------------------------------------------
 * Dequantise-then-attend (Section 3.3).  For request b and KV head h the logical cache is the
 * concatenation, in block-table order, of the pages of the row; a page with tag 0 (Recent) or
 * 1 (Anchor) is an FP8 record of the FP8 arena, tag 2 (Stale) a TQ3 record of the TQ3 arena.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    const uint8_t* fp8_arena;
    const uint8_t* tq3_arena;
    int64_t fp8_pages, tq3_pages;
    int d, hkv, group;
    int M;                      /* 16-token tiles per page (page = 16 M tokens) */
    float k_scale, v_scale;
    const int8_t* sigma;
} orc_pool;

/* materialise K^ and V^ (fp64, [len][d]) of one (request row, kv head); returns 0 or -1 on a
 * bad tag / id */
static int materialise(const orc_pool* p, const int32_t* row, const uint8_t* tags, int len, int h,
                       double* K, double* V)
{
    int d = p->d, M = p->M, T = ORC_T * M, n_pages = (len + T - 1) / T, pg, t, i;
    uint8_t* kc = (uint8_t*)malloc((size_t)T * d);
    uint8_t* vc = (uint8_t*)malloc((size_t)T * d);
    uint16_t* g = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)T);
    uint16_t sc[ORC_MAXD], zp[ORC_MAXD];
    int rc = 0;
    for (pg = 0; pg < n_pages && rc == 0; ++pg) {
        int valid = len - pg * T < T ? len - pg * T : T;
        int64_t id = row[pg];
        if (tags[pg] <= 1) {
            const uint8_t* blk;
            if (id < 0 || id >= p->fp8_pages) { rc = -1; break; }
            blk = p->fp8_arena + (id * p->hkv + h) * orc_fp8_block_bytes(d, M);
            for (t = 0; t < valid; ++t) {
                const uint8_t* rec = blk + (int64_t)(t / ORC_T) * orc_fp8_record_bytes(d);   /* tile of the token */
                int s = t % ORC_T;
                for (i = 0; i < d; ++i) {
                    K[((int64_t)pg * T + t) * d + i] = orc_e4m3_decode(rec[s * d + i]) * (double)p->k_scale;
                    V[((int64_t)pg * T + t) * d + i] = orc_e4m3_decode(rec[16 * d + i * ORC_T + s]) * (double)p->v_scale;
                }
            }
        } else if (tags[pg] == 2) {
            const uint8_t* blk;
            if (id < 0 || id >= p->tq3_pages || valid != T) { rc = -1; break; }
            blk = p->tq3_arena + (id * p->hkv + h) * orc_tq3_block_bytes(d, M);
            orc_tq3_unpack_block(d, M, blk, kc, g, vc, sc, zp);
            for (t = 0; t < T; ++t) {
                orc_tq3_decode_key(kc + (int64_t)t * d, g[t], d, p->sigma, K + ((int64_t)pg * T + t) * d);
                for (i = 0; i < d; ++i)
                    V[((int64_t)pg * T + t) * d + i] = orc_tq3_decode_value(vc[(int64_t)t * d + i], sc[i], zp[i]);
            }
        } else {
            rc = -1;
        }
    }
    free(kc); free(vc); free(g);
    return rc;
}

/* softmax(scale * q K^T) V over tokens [lo, hi) of a materialised cache, two passes.
 * Returns the partition's maximum m, exponential sum l and NORMALISED output O (Section 3.3:
 * O_j = l_j^-1 sum_i exp(s_i - m_j) v_i).  An empty range gives m = -inf, l = 0, O = 0. */
static void attend_range(const double* q, const double* K, const double* V, int d, int lo, int hi,
                         double scale, double* m_out, double* l_out, double* O)
{
    double m = -INFINITY, l = 0.0;
    int i, c;
    for (c = 0; c < d; ++c) O[c] = 0.0;
    for (i = lo; i < hi; ++i) {
        double s = 0.0;
        for (c = 0; c < d; ++c) s += q[c] * K[(int64_t)i * d + c];
        s *= scale;
        if (s > m) m = s;
    }
    for (i = lo; i < hi; ++i) {
        double s = 0.0, w;
        for (c = 0; c < d; ++c) s += q[c] * K[(int64_t)i * d + c];
        s *= scale;
        w = exp(s - m);
        l += w;
        for (c = 0; c < d; ++c) O[c] += w * V[(int64_t)i * d + c];
    }
    if (l > 0.0)
        for (c = 0; c < d; ++c) O[c] /= l;
    *m_out = m;
    *l_out = l;
}

/* Decode attention for the newest position of every request.
 *   q bf16 bits [B][Hq][d], block_table int32 [B][max_pages], tier_tag uint8 [B][max_pages],
 *   seq_lens int32 [B]; out fp64 [B][Hq][d]; lse fp64 [B][Hq] (may be NULL).
 *   query head hq reads KV head hq / group.  seq_len 0 -> out row 0, lse -inf.
 *   mode 0: one softmax over the whole concatenated cache (the definition).
 *   mode 1: Eq. (softmax-merge): the tokens are partitioned by FORMAT (FP8 tokens, TQ3 tokens),
 *           each partition reports (m_j, l_j, normalised O_j) and the partitions are merged.
 *   mode >= 2: Eq. (softmax-merge) over `mode` contiguous token ranges of equal size.
 *   only_b / only_h >= 0 restrict the work to one request / one KV head (other outputs untouched).
 * Returns 0, or -1 if a table entry is invalid. */
int orc_decode_attention_blocks(const uint8_t* fp8_arena, int64_t fp8_pages, const uint8_t* tq3_arena,
                                int64_t tq3_pages, int d, int hkv, int group, int M, float k_scale, float v_scale,
                                const int8_t* sigma, const uint16_t* q, const int32_t* block_table,
                                const uint8_t* tier_tag, const int32_t* seq_lens, int B, int max_pages,
                                double scale, double* out, double* lse, int mode, int only_b, int only_h)
{
    orc_pool pool;
    int Hq = hkv * group, unit, rc = 0;
    pool.fp8_arena = fp8_arena; pool.tq3_arena = tq3_arena;
    pool.fp8_pages = fp8_pages; pool.tq3_pages = tq3_pages;
    pool.d = d; pool.hkv = hkv; pool.group = group; pool.M = M;
    pool.k_scale = k_scale; pool.v_scale = v_scale; pool.sigma = sigma;
    if (M < 1) return -1;

#pragma omp parallel for schedule(dynamic, 1)
    for (unit = 0; unit < B * hkv; ++unit) {
        int b = unit / hkv, h = unit % hkv, len = seq_lens[b], gq, c, j;
        const int32_t* row = block_table + (int64_t)b * max_pages;
        const uint8_t* tags = tier_tag + (int64_t)b * max_pages;
        double *K, *V, qd[ORC_MAXD], O[ORC_MAXD], Oj[ORC_MAXD];
        if ((only_b >= 0 && b != only_b) || (only_h >= 0 && h != only_h)) continue;
        if (len <= 0) {
            for (gq = 0; gq < group; ++gq) {
                int hq = h * group + gq;
                for (c = 0; c < d; ++c) out[((int64_t)b * Hq + hq) * d + c] = 0.0;
                if (lse) lse[(int64_t)b * Hq + hq] = -INFINITY;
            }
            continue;
        }
        K = (double*)malloc(sizeof(double) * (size_t)len * d);
        V = (double*)malloc(sizeof(double) * (size_t)len * d);
        if (materialise(&pool, row, tags, len, h, K, V) != 0) {
#pragma omp atomic write
            rc = -1;
            free(K); free(V);
            continue;
        }
        for (gq = 0; gq < group; ++gq) {
            int hq = h * group + gq;
            double m, l;
            for (c = 0; c < d; ++c) qd[c] = (double)orc_bf16_to_f32(q[((int64_t)b * Hq + hq) * d + c]);
            if (mode == 0) {
                attend_range(qd, K, V, d, 0, len, scale, &m, &l, O);
            } else {
                /* partitions: list of token index sets; here realised as gathered copies */
                int n_part = (mode == 1) ? 2 : mode;
                double* mj = (double*)malloc(sizeof(double) * n_part);
                double* lj = (double*)malloc(sizeof(double) * n_part);
                double* Oall = (double*)malloc(sizeof(double) * (size_t)n_part * d);
                double acc;
                for (j = 0; j < n_part; ++j) {
                    if (mode == 1) {
                        /* gather the tokens whose page has format j (0 = FP8, 1 = TQ3) */
                        double* Kp = (double*)malloc(sizeof(double) * (size_t)len * d);
                        double* Vp = (double*)malloc(sizeof(double) * (size_t)len * d);
                        int n = 0, i;
                        for (i = 0; i < len; ++i)
                            if ((tags[i / (ORC_T * M)] == 2) == (j == 1)) {
                                memcpy(Kp + (int64_t)n * d, K + (int64_t)i * d, sizeof(double) * d);
                                memcpy(Vp + (int64_t)n * d, V + (int64_t)i * d, sizeof(double) * d);
                                ++n;
                            }
                        attend_range(qd, Kp, Vp, d, 0, n, scale, &mj[j], &lj[j], Oj);
                        free(Kp); free(Vp);
                    } else {
                        int lo = (int)((int64_t)len * j / n_part), hi = (int)((int64_t)len * (j + 1) / n_part);
                        attend_range(qd, K, V, d, lo, hi, scale, &mj[j], &lj[j], Oj);
                    }
                    memcpy(Oall + (int64_t)j * d, Oj, sizeof(double) * d);
                }
                /* m = max_j m_j ; l = sum_j e^{m_j - m} l_j ; O = sum_j e^{m_j-m} l_j O_j / l */
                m = -INFINITY;
                for (j = 0; j < n_part; ++j) if (mj[j] > m) m = mj[j];
                l = 0.0;
                for (j = 0; j < n_part; ++j) if (lj[j] > 0.0) l += exp(mj[j] - m) * lj[j];
                for (c = 0; c < d; ++c) {
                    acc = 0.0;
                    for (j = 0; j < n_part; ++j)
                        if (lj[j] > 0.0) acc += exp(mj[j] - m) * lj[j] * Oall[(int64_t)j * d + c];
                    O[c] = acc / l;
                }
                free(mj); free(lj); free(Oall);
            }
            for (c = 0; c < d; ++c) out[((int64_t)b * Hq + hq) * d + c] = O[c];
            if (lse) lse[(int64_t)b * Hq + hq] = m + log(l);
        }
        free(K); free(V);
    }
    return rc;
}

/* the 16-token page (M = 1) */
int orc_decode_attention(const uint8_t* fp8_arena, int64_t fp8_pages, const uint8_t* tq3_arena,
                         int64_t tq3_pages, int d, int hkv, int group, float k_scale, float v_scale,
                         const int8_t* sigma, const uint16_t* q, const int32_t* block_table,
                         const uint8_t* tier_tag, const int32_t* seq_lens, int B, int max_pages,
                         double scale, double* out, double* lse, int mode, int only_b, int only_h)
{
    return orc_decode_attention_blocks(fp8_arena, fp8_pages, tq3_arena, tq3_pages, d, hkv, group, 1, k_scale, v_scale,
                                       sigma, q, block_table, tier_tag, seq_lens, B, max_pages, scale, out, lse, mode,
                                       only_b, only_h);
}

/* ------------------------------------------------------------------------------------------
 * Globally normalised page mass (Section 3.1, Eq. score-partial, Eq. score-global-weight,
 * Eq. attention-score).  For query head h the tokens are split into partitions j by physical
 * FORMAT (j = 0: FP8 pages, j = 1: TQ3 pages), each partition reports
 *      m_j = max_{i in j} s_i,   l_j = sum_{i in j} e^{s_i - m_j},
 * with m = max_j m_j and l = sum_j e^{m_j - m} l_j; a page p of partition j has
 *      rho_p = (1 / l_j) sum_{i in p} e^{s_i - m_j},   w_j = e^{m_j - m} l_j / l,
 *      q_p = w_j rho_p,   q~_p = q_p / sum_p' q_p'   (no sink state here: every page is addressable).
 * mass[b][hq][p] receives q~ (0 for pages beyond the request's length).
 * Returns 0, or -1 if a table entry is invalid. */
int orc_page_mass_blocks(const uint8_t* fp8_arena, int64_t fp8_pages, const uint8_t* tq3_arena, int64_t tq3_pages,
                         int d, int hkv, int group, int M, float k_scale, float v_scale, const int8_t* sigma,
                         const uint16_t* q, const int32_t* block_table, const uint8_t* tier_tag,
                         const int32_t* seq_lens, int B, int max_pages, double scale, double* mass)
{
    orc_pool pool;
    int Hq = hkv * group, unit, rc = 0, T = ORC_T * M;      /* pages of T = 16 M tokens */
    pool.fp8_arena = fp8_arena; pool.tq3_arena = tq3_arena;
    pool.fp8_pages = fp8_pages; pool.tq3_pages = tq3_pages;
    pool.d = d; pool.hkv = hkv; pool.group = group; pool.M = M;
    pool.k_scale = k_scale; pool.v_scale = v_scale; pool.sigma = sigma;
    if (M < 1) return -1;

#pragma omp parallel for schedule(dynamic, 1)
    for (unit = 0; unit < B * hkv; ++unit) {
        int b = unit / hkv, h = unit % hkv, len = seq_lens[b], gq, c, i, pg, j;
        int n_pages = len > 0 ? (len + T - 1) / T : 0;
        const int32_t* row = block_table + (int64_t)b * max_pages;
        const uint8_t* tags = tier_tag + (int64_t)b * max_pages;
        double *K, *V, *s;
        for (gq = 0; gq < group; ++gq)
            for (pg = 0; pg < max_pages; ++pg) mass[((int64_t)b * Hq + h * group + gq) * max_pages + pg] = 0.0;
        if (len <= 0) continue;
        K = (double*)malloc(sizeof(double) * (size_t)len * d);
        V = (double*)malloc(sizeof(double) * (size_t)len * d);
        s = (double*)malloc(sizeof(double) * (size_t)len);
        if (materialise(&pool, row, tags, len, h, K, V) != 0) {
#pragma omp atomic write
            rc = -1;
            free(K); free(V); free(s);
            continue;
        }
        for (gq = 0; gq < group; ++gq) {
            int hq = h * group + gq;
            double* out = mass + ((int64_t)b * Hq + hq) * max_pages;
            double mj[2] = {-INFINITY, -INFINITY}, lj[2] = {0.0, 0.0}, m, l, total = 0.0;
            for (i = 0; i < len; ++i) {
                double acc = 0.0;
                for (c = 0; c < d; ++c)
                    acc += (double)orc_bf16_to_f32(q[((int64_t)b * Hq + hq) * d + c]) * K[(int64_t)i * d + c];
                s[i] = scale * acc;
                j = tags[i / T] == 2;
                if (s[i] > mj[j]) mj[j] = s[i];
            }
            for (i = 0; i < len; ++i) {
                j = tags[i / T] == 2;
                lj[j] += exp(s[i] - mj[j]);
            }
            m = mj[0] > mj[1] ? mj[0] : mj[1];
            l = 0.0;
            for (j = 0; j < 2; ++j) if (lj[j] > 0.0) l += exp(mj[j] - m) * lj[j];
            for (pg = 0; pg < n_pages; ++pg) {
                int lo = pg * T, hi = lo + T < len ? lo + T : len;
                double rho = 0.0, w;
                j = tags[pg] == 2;
                for (i = lo; i < hi; ++i) rho += exp(s[i] - mj[j]);
                rho /= lj[j];
                w = exp(mj[j] - m) * lj[j] / l;
                out[pg] = w * rho;
                total += out[pg];
            }
            for (pg = 0; pg < n_pages; ++pg) out[pg] /= total;
        }
        free(K); free(V); free(s);
    }
    return rc;
}

int orc_page_mass(const uint8_t* fp8_arena, int64_t fp8_pages, const uint8_t* tq3_arena, int64_t tq3_pages,
                  int d, int hkv, int group, float k_scale, float v_scale, const int8_t* sigma,
                  const uint16_t* q, const int32_t* block_table, const uint8_t* tier_tag,
                  const int32_t* seq_lens, int B, int max_pages, double scale, double* mass)
{
    return orc_page_mass_blocks(fp8_arena, fp8_pages, tq3_arena, tq3_pages, d, hkv, group, 1, k_scale, v_scale, sigma, q,
                                block_table, tier_tag, seq_lens, B, max_pages, scale, mass);
}

/* Eq. (attention-score): r_p = mean over the sampled head set of q~_{h,p}; a_p <- beta a_p + (1 - beta) r_p.
 * head_mask bit hq selects query head hq (at least one bit set among the first Hq).  mass is
 * [B][Hq][max_pages], score is [B][max_pages] and is updated in place for pages below the length. */
void orc_page_score_update_blocks(const double* mass, const int32_t* seq_lens, int B, int Hq, int max_pages,
                                  int page_tokens, uint64_t head_mask, double beta, double* score)
{
    int b, pg, hq, n_heads = 0;
    for (hq = 0; hq < Hq; ++hq) if ((head_mask >> hq) & 1u) ++n_heads;
    for (b = 0; b < B; ++b) {
        int n_pages = seq_lens[b] > 0 ? (seq_lens[b] + page_tokens - 1) / page_tokens : 0;
        for (pg = 0; pg < n_pages; ++pg) {
            double r = 0.0;
            for (hq = 0; hq < Hq; ++hq)
                if ((head_mask >> hq) & 1u) r += mass[((int64_t)b * Hq + hq) * max_pages + pg];
            r /= (double)n_heads;
            score[(int64_t)b * max_pages + pg] = beta * score[(int64_t)b * max_pages + pg] + (1.0 - beta) * r;
        }
    }
}

void orc_page_score_update(const double* mass, const int32_t* seq_lens, int B, int Hq, int max_pages,
                           uint64_t head_mask, double beta, double* score)
{
    orc_page_score_update_blocks(mass, seq_lens, B, Hq, max_pages, ORC_T, head_mask, beta, score);
}

/* ------------------------------------------------------------------------------------------
 * Byte accounting (Eq. kv-per-token, Eq. effective-bits, Section 6.3 counters).
 * page = T tokens; the TQ3 structure per page and KV head is
 *    K: T * 3d/8 bytes of codes + T * 2 bytes fp16 norm correction (per token)
 *    V: T * 3d/8 bytes of codes + d * (2+2) bytes fp16 scale and zero (per channel, per page)
 * ---------------------------------------------------------------------------------------- */
int64_t orc_kv_bytes_per_token(int layers, int hkv, int d, int bytes_per_scalar)
{
    return 2 * (int64_t)layers * hkv * d * bytes_per_scalar;
}

int64_t orc_page_bytes_dense(int T, int d, int hkv, int bytes_per_scalar)
{
    return 2 * (int64_t)T * d * hkv * bytes_per_scalar;
}

int64_t orc_page_bytes_tq3(int T, int d, int hkv)
{
    int64_t kpart = (int64_t)T * (3 * d / 8) + (int64_t)T * 2;
    int64_t vpart = (int64_t)T * (3 * d / 8) + (int64_t)d * 4;
    return hkv * (kpart + vpart);
}

/* realised physical TQ3 rate b_S in bits per scalar, metadata included */
double orc_tq3_bits_per_scalar(int T, int d)
{
    return 8.0 * (double)orc_page_bytes_tq3(T, d, 1) / (2.0 * T * d);
}

/* b_eff = 8 (p_R + p_A) + b_S p_S + b_meta */
double orc_effective_bits(double p_R, double p_A, double p_S, double b_S, double b_meta)
{
    return 8.0 * (p_R + p_A) + b_S * p_S + b_meta;
}

/* ------------------------------------------------------------------------------------------
 * Bulk helper: write every page of one request into the arenas.
 *   k_bits, v_bits: bf16 bit patterns [len][hkv][d] (token-major, as handed to Append)
 *   row[pg], tags[pg]: physical id and tier tag of logical page pg
 *   Recent/Anchor pages: bf16 -> e4m3 (a partial last page keeps zero bytes in unused slots);
 *   Stale pages: TQ3 encoded from the bf16 originals (must be full).
 * Returns 0, or -1 on an invalid tag or a partial Stale page.
 * ---------------------------------------------------------------------------------------- */
int orc_encode_request_blocks(int d, int hkv, int len, int M, const uint16_t* k_bits, const uint16_t* v_bits,
                              const int32_t* row, const uint8_t* tags, const int8_t* sigma, float k_scale,
                              float v_scale, uint8_t* fp8_arena, uint8_t* tq3_arena)
{
    int T = ORC_T * M, n_pages = (len + T - 1) / T, pg, rc = 0;
#pragma omp parallel for schedule(dynamic, 8)
    for (pg = 0; pg < n_pages; ++pg) {
        int valid = len - pg * T < T ? len - pg * T : T, h, t, i;
        float* k = (float*)malloc(sizeof(float) * (size_t)T * d);
        float* v = (float*)malloc(sizeof(float) * (size_t)T * d);
        for (h = 0; h < hkv; ++h) {
            memset(k, 0, sizeof(float) * (size_t)T * d);
            memset(v, 0, sizeof(float) * (size_t)T * d);
            for (t = 0; t < valid; ++t)
                for (i = 0; i < d; ++i) {
                    int64_t src = (((int64_t)pg * T + t) * hkv + h) * d + i;
                    k[(int64_t)t * d + i] = orc_bf16_to_f32(k_bits[src]);
                    v[(int64_t)t * d + i] = orc_bf16_to_f32(v_bits[src]);
                }
            if (tags[pg] <= 1) {
                orc_fp8_pack_block(d, M, k, v, valid, k_scale, v_scale,
                                   fp8_arena + ((int64_t)row[pg] * hkv + h) * orc_fp8_block_bytes(d, M));
            } else if (tags[pg] == 2 && valid == T) {
                orc_tq3_block_from_f32(d, M, k, v, sigma,
                                       tq3_arena + ((int64_t)row[pg] * hkv + h) * orc_tq3_block_bytes(d, M));
            } else {
#pragma omp atomic write
                rc = -1;
            }
        }
        free(k); free(v);
    }
    return rc;
}

int orc_encode_request(int d, int hkv, int len, const uint16_t* k_bits, const uint16_t* v_bits,
                       const int32_t* row, const uint8_t* tags, const int8_t* sigma, float k_scale,
                       float v_scale, uint8_t* fp8_arena, uint8_t* tq3_arena)
{
    return orc_encode_request_blocks(d, hkv, len, 1, k_bits, v_bits, row, tags, sigma, k_scale, v_scale, fp8_arena,
                                     tq3_arena);
}

/* ------------------------------------------------------------------------------------------
 * Promote(p) of Algorithm 1, data part: reconstruct a TQ3 record into an FP8 record.
 * The reconstruction is specified in fp32 with a fixed operation order (so that it can be
 * reproduced bit for bit), then rounded to e4m3 like Append:
 *   key   : y = H c (butterflies, strides ascending, c = signed fp16 levels as fp32);
 *           k = sigma .* ((g * rs) * y), rs = fp32(1/sqrt(d));   stored = e4m3(k * (1/k_scale))
 *   value : v = sc * code + zp as one multiplication and one addition; stored = e4m3(v * (1/v_scale))
 * ---------------------------------------------------------------------------------------- */
void orc_promote_record(int d, const uint8_t* tq3_rec, float k_scale, float v_scale, const int8_t* sigma,
                        uint8_t* fp8_rec)
{
    uint8_t* kc = (uint8_t*)malloc(ORC_T * (size_t)d);
    uint8_t* vc = (uint8_t*)malloc(ORC_T * (size_t)d);
    uint16_t g[ORC_T], sc[ORC_MAXD], zp[ORC_MAXD];
    float ik = 1.0f / k_scale, iv = 1.0f / v_scale, rs = (float)(1.0 / sqrt((double)d));
    int t, i, h;
    orc_tq3_unpack_record(d, tq3_rec, kc, g, vc, sc, zp);
    memset(fp8_rec, 0, (size_t)orc_fp8_record_bytes(d));
    for (t = 0; t < ORC_T; ++t) {
        float y[ORC_MAXD], gr = orc_f16_to_f32(g[t]) * rs;
        for (i = 0; i < d; ++i) {
            float c = ORC_C[kc[t * d + i] & 3];
            y[i] = (kc[t * d + i] & 4) ? -c : c;
        }
        for (h = 1; h < d; h <<= 1)
            for (i = 0; i < d; ++i)
                if ((i & h) == 0) {
                    float u = y[i], w = y[i + h];
                    y[i] = u + w;
                    y[i + h] = u - w;
                }
        for (i = 0; i < d; ++i) {
            float k = gr * y[i];
            if (sigma[i] < 0) k = -k;
            fp8_rec[t * d + i] = orc_e4m3_encode(k * ik);
        }
    }
    for (i = 0; i < d; ++i) {
        float s = orc_f16_to_f32(sc[i]), z = orc_f16_to_f32(zp[i]);
        for (t = 0; t < ORC_T; ++t) {
            float p = s * (float)vc[t * d + i];
            float v = p + z;
            fp8_rec[16 * d + i * ORC_T + t] = orc_e4m3_encode(v * iv);
        }
    }
    free(kc); free(vc);
}
