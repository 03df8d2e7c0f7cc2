/*
 * CPU oracle for AdaComp pack() and unpack()-and-sum.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow restatement of Algorithm 2 ("Details of pack()")
 * and of the unpack()/sum half of Algorithm 1 of the AdaComp paper, in IEEE
 * binary32 (the precision the method is stated in), written to be checked
 * against the paper by eye.  It shares no code with the CUDA library and is
 * only ever called from the tests, from the smoke check and from the
 * benchmark's CPU-baseline leg.  Build: gcc -O2 -ffp-contract=off (no fast-math),
 * so every add/sub is a single rounded binary32 operation and denormals are kept.
 *
 * Parity pins: hand-worked bins, closed-form special cases, brute force against
 * an independent scalar Python restatement, and exact-sum checks against
 * rational arithmetic live in the CPU test-suite.  No function here is unpinned.
 *
 * Where the paper is silent the following readings are taken (each is tested):
 *   - the last bin may be short (Section 2.5 says Algorithm 2 assumes T | length);
 *   - g_max(i) is the largest |G| in bin i (Algorithm 2, "largest absolute value");
 *   - an element is sent when |H| >= g_max(i) (Algorithm 2) or when it IS the
 *     bin maximum (Section 2.4 describes the other residues as sent in addition
 *     to the maximum); flag bit 0 drops the second clause (literal Algorithm 2);
 *   - bins whose maximum is zero send nothing, and an element with G == 0 is
 *     never sent (its ternary value would be 0);
 *   - Quantize(G) = sign(G) * scale, scale = mean over ALL bins of g_max
 *     (Section 2.5), the sum taken exactly, rounded once to double, divided by
 *     the bin count in double and rounded to binary32;
 *   - the wire word is (index_in_bin << 2) | code with code 01 = +scale and
 *     11 = -scale, 8 bits wide for L_T <= 64 and 16 bits up to L_T = 16384
 *     (Section "Experiment Results": 8-/16-bit sparse-indexed words, 2 bits of
 *     which hold the ternary value);
 *   - unpack() scatters +-scale_l; the sum over learners runs l = 0..k-1 in
 *     order starting from +0.0f.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAGIC 0x31434441u /* "ADC1" little-endian */
#define ORACLE_HEADER_BYTES 64u

static uint64_t align16(uint64_t x) { return (x + 15u) & ~(uint64_t)15u; }

/* ---- stream geometry: a pure function of (n, L_T) ------------------------ */

typedef struct {
    uint32_t w;          /* bytes per word */
    uint32_t tile_bins;  /* bins per directory tile */
    uint64_t n_bins;
    uint64_t n_tiles;
    uint64_t tile_off_at; /* byte offsets of the sections */
    uint64_t bin_cnt_at;
    uint64_t payload_at;
} geometry;

static geometry geometry_of(uint64_t n, uint32_t L_T)
{
    geometry g;
    g.w = (L_T <= 64u) ? 1u : 2u;
    g.tile_bins = (L_T <= 1000u) ? 4u * (1000u / L_T) : 1u;
    g.n_bins = (n + L_T - 1u) / L_T;
    g.n_tiles = (g.n_bins + g.tile_bins - 1u) / g.tile_bins;
    g.tile_off_at = ORACLE_HEADER_BYTES;
    g.bin_cnt_at = align16(g.tile_off_at + 8u * (g.n_tiles + 1u));
    g.payload_at = align16(g.bin_cnt_at + g.n_bins * g.w);
    return g;
}

uint64_t adacomp_oracle_stream_bytes(uint64_t n, uint32_t L_T, uint64_t n_sel)
{
    geometry g = geometry_of(n, L_T);
    return g.payload_at + align16(n_sel * g.w);
}

/* ---- little-endian field access ------------------------------------------ */

static void put_u16(uint8_t *p, uint16_t v) { p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); }
static void put_u32(uint8_t *p, uint32_t v) { for (int i = 0; i < 4; i++) p[i] = (uint8_t)(v >> (8 * i)); }
static void put_u64(uint8_t *p, uint64_t v) { for (int i = 0; i < 8; i++) p[i] = (uint8_t)(v >> (8 * i)); }
static uint16_t get_u16(const uint8_t *p) { return (uint16_t)(p[0] | (p[1] << 8)); }
static uint32_t get_u32(const uint8_t *p) { uint32_t v = 0; for (int i = 3; i >= 0; i--) v = (v << 8) | p[i]; return v; }
static uint64_t get_u64(const uint8_t *p) { uint64_t v = 0; for (int i = 7; i >= 0; i--) v = (v << 8) | p[i]; return v; }

/* ---- exact sum of non-negative binary32 values --------------------------- */
/*
 * Every finite binary32 value is an integer multiple of 2^-149 below 2^128,
 * so a 320-bit unsigned integer holds the exact sum of up to 2^31 of them.
 * The sum is then rounded once, to nearest-even, to a double.
 */
#define BIG_LIMBS 10

static void big_add_f32(uint32_t limb[BIG_LIMBS], float v)
{
    uint32_t bits;
    memcpy(&bits, &v, 4);
    uint32_t e = (bits >> 23) & 0xffu;
    uint32_t frac = bits & 0x7fffffu;
    uint64_t m = e ? (frac | 0x800000u) : frac;   /* value = m * 2^(shift-149) */
    uint32_t shift = e ? e - 1u : 0u;
    uint32_t at = shift / 32u;
    uint64_t add = m << (shift % 32u);            /* < 2^55 */
    uint64_t carry = 0;
    for (uint32_t i = at; i < BIG_LIMBS && (add || carry); i++) {
        uint64_t s = (uint64_t)limb[i] + (add & 0xffffffffu) + carry;
        limb[i] = (uint32_t)s;
        carry = s >> 32;
        add >>= 32;
    }
}

static int big_bit(const uint32_t limb[BIG_LIMBS], int pos)
{
    return (limb[pos / 32] >> (pos % 32)) & 1u;
}

static double big_to_double_units(const uint32_t limb[BIG_LIMBS])
{
    /* returns the double nearest to (integer value) * 2^-149 */
    int top = -1;
    for (int pos = 32 * BIG_LIMBS - 1; pos >= 0; pos--)
        if (big_bit(limb, pos)) { top = pos; break; }
    if (top < 0) return 0.0;
    uint64_t mant = 0;
    int low = top - 52;               /* position of the last kept bit */
    if (low <= 0) {
        for (int pos = top; pos >= 0; pos--) mant = (mant << 1) | (uint64_t)big_bit(limb, pos);
        return ldexp((double)mant, -149);
    }
    for (int pos = top; pos >= low; pos--) mant = (mant << 1) | (uint64_t)big_bit(limb, pos);
    int round_bit = big_bit(limb, low - 1);
    int sticky = 0;
    for (int pos = low - 2; pos >= 0 && !sticky; pos--) sticky = big_bit(limb, pos);
    if (round_bit && (sticky || (mant & 1u))) mant += 1;   /* ties to even */
    return ldexp((double)mant, low - 149);
}

/* exposed so the tests can pin the summation by itself against rational arithmetic */
double adacomp_oracle_exact_sum(const float *v, uint64_t count)
{
    uint32_t limb[BIG_LIMBS] = {0};
    for (uint64_t i = 0; i < count; i++) big_add_f32(limb, v[i]);
    return big_to_double_units(limb);
}

/* ---- pack(): Algorithm 2 -------------------------------------------------- */

/*
 * Threads the per-element and per-bin loops of pack() may use (default 1: the checker the tests
 * pin).  Every bin is worked on its own and the sum of the bin maxima is exact, so the stream and
 * the residue do not depend on this number; the benchmark's all-host-cores baseline sets it.
 */
static int oracle_threads = 1;

void adacomp_oracle_set_threads(int threads) { oracle_threads = threads > 1 ? threads : 1; }
int adacomp_oracle_get_threads(void) { return oracle_threads; }

/*
 * Which elements of one bin are sent (Algorithm 2's test inside its second pair of loops, with the
 * readings listed at the top of this file).  The bin holds elements [lo, hi) of the layer and
 * `largest` is its g_max.  The places of the sent elements inside the bin are written to `places`
 * (ascending; skipped when NULL); the return value is how many there are.
 */
static uint32_t sent_places_of_bin(const float *G, const float *H, uint64_t lo, uint64_t hi, float largest,
                                   int literal, uint16_t *places)
{
    uint32_t sent = 0;
    if (!(largest > 0.0f)) return 0;                 /* a bin of zeros sends nothing */
    for (uint64_t i = lo; i < hi; i++) {
        if (G[i] == 0.0f) continue;                  /* its ternary value would be 0 */
        const int passes_test = fabsf(H[i]) >= largest;
        const int is_the_maximum = !literal && fabsf(G[i]) == largest;
        if (passes_test || is_the_maximum) {
            if (places) places[sent] = (uint16_t)(i - lo);
            sent++;
        }
    }
    return sent;
}

/*
 * dW[n] in; residue[n] in/out; out[out_cap] receives the stream.
 * g_max_out (optional, n_bins floats) receives the bin maxima.
 * Returns 0, or -1 bad argument, -2 out of memory, -3 out_cap too small.
 *
 * `factor`: the multiplier of the latest gradient in the selection test (Section 2.4 studies 1.5 to
 * 3.0 and settles on 2 because it needs additions only).  0 selects the paper's choice as
 * Algorithm 2 writes it, H = G + dW with two additions; any other value takes the general form
 * H = residue + factor * dW, one rounded multiplication and one rounded addition (for factor 2 the
 * two forms can differ in the last place, which is why they are kept apart).  Factor 1 makes H = G:
 * only the bin maxima are sent, which is the local selection without the soft threshold that the
 * paper compares against (Section 5, "LS").  Streams made with a factor carry bit 1 in the header's flags.
 *
 * `quantiser`: Section 2.5 notes that the method is not tied to one quantisation function.  0 is the
 * paper's: sign(G) times the average of the g_max vector over all bins.  1 keeps the sign and the one value
 * per layer but takes for it the average |G| of the elements that are sent (the value that makes the
 * squared error of the sent elements smallest): the exact sum of those |G|, rounded once to double,
 * divided by their number in double and rounded to binary32; 0 when nothing is sent.  The selection does
 * not depend on the quantiser.  Streams made with quantiser 1 carry bit 2 in the header's flags.
 */
int adacomp_oracle_pack_general(const float *dW, float *residue, uint64_t n, uint32_t L_T, uint32_t flags,
                                float factor, uint32_t quantiser, uint8_t *out, uint64_t out_cap, float *g_max_out);

int adacomp_oracle_pack_scaled(const float *dW, float *residue, uint64_t n, uint32_t L_T,
                               uint32_t flags, float factor, uint8_t *out, uint64_t out_cap, float *g_max_out)
{
    return adacomp_oracle_pack_general(dW, residue, n, L_T, flags, factor, 0u, out, out_cap, g_max_out);
}

int adacomp_oracle_pack(const float *dW, float *residue, uint64_t n, uint32_t L_T,
                        uint32_t flags, uint8_t *out, uint64_t out_cap, float *g_max_out)
{
    return adacomp_oracle_pack_scaled(dW, residue, n, L_T, flags, 0.0f, out, out_cap, g_max_out);
}

int adacomp_oracle_pack_general(const float *dW, float *residue, uint64_t n, uint32_t L_T, uint32_t flags,
                                float factor, uint32_t quantiser, uint8_t *out, uint64_t out_cap, float *g_max_out)
{
    if (L_T == 0 || L_T > 16384u || !out || (n && (!dW || !residue))) return -1;
    if (factor != 0.0f && !(factor > 0.0f && factor <= 1e30f)) return -1;
    if (quantiser > 1u) return -1;
    flags = (flags & 1u) | (factor != 0.0f ? 2u : 0u) | (quantiser == 1u ? 4u : 0u);
    const int literal = (flags & 1u) != 0;
    const int threads = oracle_threads;
    (void)threads;
    geometry geo = geometry_of(n, L_T);
    if (out_cap < geo.payload_at) return -3;
    const int64_t bins = (int64_t)geo.n_bins, elems = (int64_t)n;

    float *G = (float *)malloc((n ? n : 1) * sizeof(float));
    float *H = (float *)malloc((n ? n : 1) * sizeof(float));
    float *g_max = (float *)malloc((geo.n_bins ? geo.n_bins : 1) * sizeof(float));
    uint64_t *first_word = (uint64_t *)malloc((geo.n_bins + 1u) * sizeof(uint64_t));
    if (!G || !H || !g_max || !first_word) { free(G); free(H); free(g_max); free(first_word); return -2; }

    /* G <- residue + dW ;  H <- G + dW   (two rounded additions), or H <- residue + factor * dW */
#pragma omp parallel for num_threads(threads) if (threads > 1)
    for (int64_t i = 0; i < elems; i++) {
        G[i] = residue[i] + dW[i];
        if (factor == 0.0f) {
            H[i] = G[i] + dW[i];
        } else {
            const float scaled = factor * dW[i];
            H[i] = residue[i] + scaled;
        }
    }

    /* g_max: the largest |G| of every bin */
#pragma omp parallel for num_threads(threads) if (threads > 1)
    for (int64_t b = 0; b < bins; b++) {
        uint64_t lo = (uint64_t)b * L_T, hi = lo + L_T < n ? lo + L_T : n;
        float m = 0.0f;
        for (uint64_t i = lo; i < hi; i++)
            if (fabsf(G[i]) > m) m = fabsf(G[i]);
        g_max[b] = m;
        if (g_max_out) g_max_out[b] = m;
    }

    /* one scale for the layer: the average of the g_max vector */
    float scale = 0.0f;
    if (geo.n_bins) {
        double S = adacomp_oracle_exact_sum(g_max, geo.n_bins);
        scale = (float)(S / (double)geo.n_bins);
    }

    /* how many elements each bin sends, hence where its words start in the stream */
#pragma omp parallel for num_threads(threads) if (threads > 1)
    for (int64_t b = 0; b < bins; b++) {
        uint64_t lo = (uint64_t)b * L_T, hi = lo + L_T < n ? lo + L_T : n;
        first_word[b + 1] = sent_places_of_bin(G, H, lo, hi, g_max[b], literal, NULL);
    }
    first_word[0] = 0;
    for (uint64_t b = 0; b < geo.n_bins; b++) first_word[b + 1] += first_word[b];
    const uint64_t n_sel = first_word[geo.n_bins];
    const uint64_t bytes_used = geo.payload_at + align16(n_sel * geo.w);
    const int overflow = bytes_used > out_cap;

    if (quantiser == 1u) {
        /* the other quantiser: the average |G| of the elements that are sent */
        scale = 0.0f;
        if (n_sel) {
            float *sent_abs = (float *)malloc(n_sel * sizeof(float));
            if (!sent_abs) { free(G); free(H); free(g_max); free(first_word); return -2; }
#pragma omp parallel for num_threads(threads) if (threads > 1)
            for (int64_t b = 0; b < bins; b++) {
                uint64_t lo = (uint64_t)b * L_T, hi = lo + L_T < n ? lo + L_T : n;
                uint16_t places[16384];
                const uint32_t sent = sent_places_of_bin(G, H, lo, hi, g_max[b], literal, places);
                for (uint32_t j = 0; j < sent; j++) sent_abs[first_word[b] + j] = fabsf(G[lo + places[j]]);
            }
            double S = adacomp_oracle_exact_sum(sent_abs, n_sel);
            scale = (float)(S / (double)n_sel);
            free(sent_abs);
        }
    }

    /* bin by bin: the counts, the words of the sent elements, and everybody's new residue */
    memset(out, 0, geo.payload_at);
    uint8_t *tile_off = out + geo.tile_off_at;
    uint8_t *bin_cnt = out + geo.bin_cnt_at;
    uint8_t *payload = out + geo.payload_at;
#pragma omp parallel for num_threads(threads) if (threads > 1)
    for (int64_t b = 0; b < bins; b++) {
        uint64_t lo = (uint64_t)b * L_T, hi = lo + L_T < n ? lo + L_T : n;
        uint16_t places[16384];
        const uint32_t sent = sent_places_of_bin(G, H, lo, hi, g_max[b], literal, places);
        if ((uint64_t)b % geo.tile_bins == 0) put_u64(tile_off + 8u * ((uint64_t)b / geo.tile_bins), first_word[b]);
        if (geo.w == 1u) bin_cnt[b] = (uint8_t)sent;
        else put_u16(bin_cnt + 2u * (uint64_t)b, (uint16_t)sent);
        for (uint64_t i = lo; i < hi; i++) residue[i] = G[i];          /* kept whole where nothing is sent */
        for (uint32_t j = 0; j < sent; j++) {
            const uint64_t i = lo + places[j];
            const int negative = signbit(G[i]) != 0;
            const float quantised = negative ? -scale : scale;          /* sign(G) times the layer's scale */
            residue[i] = G[i] - quantised;
            if (!overflow) {
                const uint32_t word = ((uint32_t)places[j] << 2) | (negative ? 3u : 1u);
                const uint64_t at = first_word[b] + j;
                if (geo.w == 1u) payload[at] = (uint8_t)word;
                else put_u16(payload + 2u * at, (uint16_t)word);
            }
        }
    }
    put_u64(tile_off + 8u * geo.n_tiles, n_sel);
    if (!overflow) memset(payload + n_sel * geo.w, 0, bytes_used - geo.payload_at - n_sel * geo.w);

    put_u32(out + 0, ORACLE_MAGIC);
    put_u16(out + 4, 1);
    out[6] = (uint8_t)geo.w;
    out[7] = (uint8_t)(flags & 7u);
    put_u32(out + 8, L_T);
    put_u32(out + 12, geo.tile_bins);
    put_u64(out + 16, n);
    put_u64(out + 24, geo.n_bins);
    put_u64(out + 32, geo.n_tiles);
    put_u64(out + 40, n_sel);
    uint32_t scale_bits;
    memcpy(&scale_bits, &scale, 4);
    put_u32(out + 48, scale_bits);
    put_u32(out + 52, 0);
    put_u64(out + 56, bytes_used);

    free(G); free(H); free(g_max); free(first_word);
    return overflow ? -3 : 0;
}

/* ---- stream version 2: the bins are told apart by a flag in the words -------- */
/*
 * The paper's rate figures count the words alone (Section "Experiment Results": 8 or 16 bits per sent
 * element), i.e. they leave out whatever tells the receiver which bin a word belongs to.  Version 1 spends a
 * count per bin on that (1 or 2 bytes per L_T elements).  Version 2 spends nothing but one of the word's two
 * spare bits: the first word of every bin carries a flag.  Layout: the 64-byte header (version field 2; bytes
 * 52..55 hold the number of bins that send nothing), the tile directory (u64 word offsets, as in version 1,
 * counted in version-2 words), the words, zero-padded to 16 bytes.  There is no count section.
 *   word = (index_in_bin << 2) | (first_of_bin << 1) | negative
 * A bin that sends nothing is one marker word with first_of_bin set and the index L_T (one past the bin), so that
 * every bin owns exactly one flagged word.  Words are 8 bits wide for L_T <= 63 (the marker's index must fit
 * 6 bits) and 16 bits up to 16383; L_T = 16384 has no version-2 form.
 */
static uint32_t v2_word_bytes(uint32_t L_T) { return L_T <= 63u ? 1u : 2u; }

uint64_t adacomp_oracle_v2_bytes(uint64_t n, uint32_t L_T, uint64_t n_words)
{
    geometry g = geometry_of(n, L_T);
    return align16(ORACLE_HEADER_BYTES + 8u * (g.n_tiles + 1u)) + align16(n_words * v2_word_bytes(L_T));
}

/* Version 1 stream in, version 2 stream out.  Returns 0, -1 bad argument, -3 out_cap too small, -4 malformed input. */
int adacomp_oracle_to_v2(const uint8_t *v1, uint8_t *out, uint64_t out_cap)
{
    if (!v1 || !out) return -1;
    if (get_u32(v1) != ORACLE_MAGIC || get_u16(v1 + 4) != 1) return -4;
    const uint32_t L_T = get_u32(v1 + 8);
    const uint64_t n = get_u64(v1 + 16), n_sel = get_u64(v1 + 40);
    if (L_T == 0 || L_T >= 16384u) return -1;
    geometry g = geometry_of(n, L_T);
    const uint32_t w2 = v2_word_bytes(L_T);
    const uint8_t *bin_cnt = v1 + g.bin_cnt_at, *words = v1 + g.payload_at;
    uint64_t empty = 0;
    for (uint64_t b = 0; b < g.n_bins; b++) empty += (g.w == 1u ? bin_cnt[b] : get_u16(bin_cnt + 2u * b)) == 0;
    const uint64_t n_words = n_sel + empty, pay2 = align16(ORACLE_HEADER_BYTES + 8u * (g.n_tiles + 1u));
    const uint64_t bytes_used = pay2 + align16(n_words * w2);
    if (bytes_used > out_cap) return -3;
    memset(out, 0, bytes_used);
    memcpy(out, v1, ORACLE_HEADER_BYTES);
    put_u16(out + 4, 2);
    out[6] = (uint8_t)w2;
    put_u32(out + 52, (uint32_t)empty);
    put_u64(out + 56, bytes_used);
    uint64_t at1 = 0, at2 = 0;
    for (uint64_t b = 0; b < g.n_bins; b++) {
        if (b % g.tile_bins == 0) put_u64(out + ORACLE_HEADER_BYTES + 8u * (b / g.tile_bins), at2);
        const uint32_t count = g.w == 1u ? bin_cnt[b] : get_u16(bin_cnt + 2u * b);
        if (count == 0) {                                       /* the marker of a bin that sends nothing */
            const uint32_t word = (L_T << 2) | 2u;
            if (w2 == 1u) out[pay2 + at2] = (uint8_t)word; else put_u16(out + pay2 + 2u * at2, (uint16_t)word);
            at2++;
        }
        for (uint32_t j = 0; j < count; j++, at1++, at2++) {
            if (at1 >= n_sel) return -4;
            const uint32_t word1 = g.w == 1u ? words[at1] : get_u16(words + 2u * at1);
            const uint32_t code = word1 & 3u;
            if (code != 1u && code != 3u) return -4;
            const uint32_t word = (word1 & ~3u) | (j == 0 ? 2u : 0u) | (code == 3u ? 1u : 0u);
            if (w2 == 1u) out[pay2 + at2] = (uint8_t)word; else put_u16(out + pay2 + 2u * at2, (uint16_t)word);
        }
    }
    put_u64(out + ORACLE_HEADER_BYTES + 8u * g.n_tiles, at2);
    return at1 == n_sel ? 0 : -4;
}

/* Version 2 stream in, version 1 stream out (the inverse of the above).  Same return codes. */
int adacomp_oracle_from_v2(const uint8_t *v2, uint8_t *out, uint64_t out_cap)
{
    if (!v2 || !out) return -1;
    if (get_u32(v2) != ORACLE_MAGIC || get_u16(v2 + 4) != 2) return -4;
    const uint32_t L_T = get_u32(v2 + 8);
    const uint64_t n = get_u64(v2 + 16), n_sel = get_u64(v2 + 40), empty = get_u32(v2 + 52);
    if (L_T == 0 || L_T >= 16384u) return -1;
    geometry g = geometry_of(n, L_T);
    const uint32_t w2 = v2_word_bytes(L_T);
    if (v2[6] != w2) return -4;
    const uint64_t pay2 = align16(ORACLE_HEADER_BYTES + 8u * (g.n_tiles + 1u)), n_words = n_sel + empty;
    const uint64_t bytes_used = g.payload_at + align16(n_sel * g.w);
    if (bytes_used > out_cap) return -3;
    memset(out, 0, bytes_used);
    memcpy(out, v2, ORACLE_HEADER_BYTES);
    put_u16(out + 4, 1);
    out[6] = (uint8_t)g.w;
    put_u32(out + 52, 0);
    put_u64(out + 56, bytes_used);
    uint8_t *tile_off = out + g.tile_off_at, *bin_cnt = out + g.bin_cnt_at, *words = out + g.payload_at;
    uint64_t at1 = 0, bin = 0;           /* `bin`: bins opened so far */
    uint32_t count = 0;
    for (uint64_t at2 = 0; at2 < n_words; at2++) {
        const uint32_t word = w2 == 1u ? v2[pay2 + at2] : get_u16(v2 + pay2 + 2u * at2);
        if (word & 2u) {                                        /* a new bin starts */
            if (bin > 0) { if (g.w == 1u) bin_cnt[bin - 1] = (uint8_t)count; else put_u16(bin_cnt + 2u * (bin - 1), (uint16_t)count); }
            if (bin >= g.n_bins) return -4;
            if (bin % g.tile_bins == 0) put_u64(tile_off + 8u * (bin / g.tile_bins), at1);
            bin++;
            count = 0;
        } else if (bin == 0) {
            return -4;
        }
        if ((word >> 2) == L_T) { if (!(word & 2u)) return -4; continue; }      /* the marker of an empty bin */
        if ((word >> 2) > L_T || at1 >= n_sel) return -4;
        const uint32_t word1 = (word & ~3u) | ((word & 1u) ? 3u : 1u);
        if (g.w == 1u) words[at1] = (uint8_t)word1; else put_u16(words + 2u * at1, (uint16_t)word1);
        at1++;
        count++;
    }
    if (bin > 0) { if (g.w == 1u) bin_cnt[bin - 1] = (uint8_t)count; else put_u16(bin_cnt + 2u * (bin - 1), (uint16_t)count); }
    put_u64(tile_off + 8u * g.n_tiles, at1);
    return (bin == g.n_bins && at1 == n_sel) ? 0 : -4;
}

/* unpack() and sum of version-2 streams, decoded from the flags alone (no counts are rebuilt): the same ordered
 * sum as adacomp_oracle_unpack_sum gives for the version-1 forms of the streams. */
int adacomp_oracle_unpack_sum_v2(const uint8_t *const *streams, uint32_t k, float *dst, uint64_t n)
{
    if (!streams || k == 0 || (n && !dst)) return -1;
    for (uint64_t i = 0; i < n; i++) dst[i] = 0.0f;
    for (uint32_t l = 0; l < k; l++) {
        const uint8_t *s = streams[l];
        if (get_u32(s) != ORACLE_MAGIC || get_u16(s + 4) != 2 || get_u64(s + 16) != n) return -4;
        const uint32_t L_T = get_u32(s + 8), w2 = v2_word_bytes(L_T);
        if (L_T == 0 || L_T >= 16384u || s[6] != w2) return -4;
        geometry g = geometry_of(n, L_T);
        const uint64_t pay2 = align16(ORACLE_HEADER_BYTES + 8u * (g.n_tiles + 1u));
        const uint64_t n_words = get_u64(s + 40) + get_u32(s + 52);
        uint32_t scale_bits = get_u32(s + 48);
        float scale;
        memcpy(&scale, &scale_bits, 4);
        uint64_t bin = 0;                /* bins opened so far: the current one is bin - 1 */
        for (uint64_t at = 0; at < n_words; at++) {
            const uint32_t word = w2 == 1u ? s[pay2 + at] : get_u16(s + pay2 + 2u * at);
            if (word & 2u) bin++;
            if (bin == 0 || bin > g.n_bins) return -4;
            const uint32_t idx = word >> 2;
            if (idx == L_T) continue;
            const uint64_t index = (bin - 1) * L_T + idx;
            if (idx > L_T || index >= n) return -4;
            if (word & 1u) dst[index] = dst[index] - scale;
            else dst[index] = dst[index] + scale;
        }
        if (bin != g.n_bins) return -4;
    }
    return 0;
}

/* ---- unpack() and sum ----------------------------------------------------- */
/*
 * dst[n] is overwritten with the sum over the k streams, taken in stream
 * order from +0.0f.  Returns 0, or -1 bad argument, -4 streams disagree on
 * (n, L_T, word size) or are malformed, -5 reserved ternary code 10 met.
 */
int adacomp_oracle_unpack_sum(const uint8_t *const *streams, uint32_t k, float *dst, uint64_t n)
{
    if (!streams || k == 0 || (n && !dst)) return -1;
    for (uint64_t i = 0; i < n; i++) dst[i] = 0.0f;
    uint32_t L_T0 = get_u32(streams[0] + 8);
    for (uint32_t l = 0; l < k; l++) {
        const uint8_t *s = streams[l];
        if (get_u32(s) != ORACLE_MAGIC || get_u16(s + 4) != 1) return -4;
        uint32_t L_T = get_u32(s + 8);
        if (L_T == 0 || L_T > 16384u || L_T != L_T0 || get_u64(s + 16) != n) return -4;
        geometry geo = geometry_of(n, L_T);
        if (s[6] != geo.w || get_u64(s + 24) != geo.n_bins) return -4;
        uint32_t scale_bits = get_u32(s + 48);
        float scale;
        memcpy(&scale, &scale_bits, 4);
        const uint8_t *bin_cnt = s + geo.bin_cnt_at;
        const uint8_t *payload = s + geo.payload_at;
        uint64_t at = 0;
        for (uint64_t b = 0; b < geo.n_bins; b++) {
            uint32_t count = geo.w == 1u ? bin_cnt[b] : get_u16(bin_cnt + 2u * b);
            for (uint32_t j = 0; j < count; j++, at++) {
                uint32_t word = geo.w == 1u ? payload[at] : get_u16(payload + 2u * at);
                uint32_t code = word & 3u;
                uint64_t index = b * L_T + (word >> 2);
                if (code == 2u) return -5;
                if (index >= n) return -4;
                if (code == 1u) dst[index] = dst[index] + scale;
                if (code == 3u) dst[index] = dst[index] - scale;
            }
        }
        if (at != get_u64(s + 40)) return -4;
    }
    return 0;
}
