/* CPU oracle, plain C twin of slim_oracle.py.
 *
 * TEST INFRASTRUCTURE ONLY: scalar loops, one element at a time, fp64 for the
 * linear layer.  It shares nothing with the CUDA library.  It exists (a) as a
 * second, independently written statement of the storage format and of
 * w-hat = s (q - z) that the NumPy oracle is cross-checked against, and (b) as
 * the CPU baseline that the benchmark times on the host cores.
 *
 * Layouts: codes uint8 [N][K]; scales, zeros fp16 [G][N] (G = K/128);
 * x fp16 [M][K]; y fp64 [M][N]; bits uint8 [G] in {1,2,3,4}.
 */
#include <stdint.h>
#include <string.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define GROUP 128

static double half_bits_to_double(uint16_t h) {
    _Float16 v;
    memcpy(&v, &h, sizeof v);
    return (double)v;
}

/* Slices (lo, w) of a b-bit code, in storage order (format definition). */
static int code_slices(int b, int lo[2], int w[2]) {
    switch (b) {
    case 1: lo[0] = 0; w[0] = 1; return 1;
    case 2: lo[0] = 0; w[0] = 2; return 1;
    case 3: lo[0] = 0; w[0] = 2; lo[1] = 2; w[1] = 1; return 2;
    case 4: lo[0] = 0; w[0] = 4; return 1;
    default: return 0;
    }
}

/* Where bit `bit` of the code q[n][k] lives: byte offset and bit-in-byte.
 * Group j at 16*N*B_j; 16-row tile t at t*256*b; unit at 256*unit; lane
 * L = 4*((n%16)/2) + c at 8*L; odd rows in the second 32-bit word; inside the
 * little-endian word, field f at bit w*f.  k - 128 j = 32 c + (32/w) u + f. */
static int locate_bit(int N, const uint8_t* bits, int n, int k, int bit, size_t* byte, int* bit_in_byte) {
    int j = k / GROUP, kk = k % GROUP, b = bits[j];
    size_t prefix = 0;
    for (int i = 0; i < j; ++i) prefix += bits[i];
    int lo[2], w[2];
    int ns = code_slices(b, lo, w);
    int unit_base = 0;
    for (int s = 0; s < ns; ++s) {
        if (bit >= lo[s] && bit < lo[s] + w[s]) {
            int nf = 32 / w[s];
            int c = kk / 32, rem = kk % 32, u = rem / nf, f = rem % nf;
            int t = n / 16, r = n % 16, lane = 4 * (r / 2) + c, half = r % 2;
            int bitpos = w[s] * f + (bit - lo[s]);
            *byte = 16 * (size_t)N * prefix + (size_t)t * 256 * b + 256 * (size_t)(unit_base + u) + 8 * lane + 4 * half + bitpos / 8;
            *bit_in_byte = bitpos % 8;
            return 0;
        }
        unit_base += w[s];
    }
    return -1;
}

size_t slim_oracle_packed_bytes(int N, int K, const uint8_t* bits) {
    size_t total = 0;
    for (int j = 0; j < K / GROUP; ++j) total += bits[j];
    return 16 * (size_t)N * total;
}

int slim_oracle_pack(const uint8_t* codes, const uint8_t* bits, uint8_t* packed, int N, int K) {
    if (K % GROUP || N % 16) return -1;
    memset(packed, 0, slim_oracle_packed_bytes(N, K, bits));
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            int b = bits[k / GROUP];
            uint8_t q = codes[(size_t)n * K + k];
            if (q >> b) return -2;
            for (int bit = 0; bit < b; ++bit) {
                if (!((q >> bit) & 1)) continue;
                size_t byte; int bib;
                if (locate_bit(N, bits, n, k, bit, &byte, &bib)) return -3;
                packed[byte] |= (uint8_t)(1u << bib);
            }
        }
    return 0;
}

int slim_oracle_unpack(const uint8_t* packed, const uint8_t* bits, uint8_t* codes, int N, int K) {
    if (K % GROUP || N % 16) return -1;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            int b = bits[k / GROUP];
            uint8_t q = 0;
            for (int bit = 0; bit < b; ++bit) {
                size_t byte; int bib;
                if (locate_bit(N, bits, n, k, bit, &byte, &bib)) return -3;
                q |= (uint8_t)(((packed[byte] >> bib) & 1u) << bit);
            }
            codes[(size_t)n * K + k] = q;
        }
    return 0;
}

/* fp16_rn( f32(s) * ( f32(q) - f32(z) ) ), both operations in IEEE single. */
void slim_oracle_dequant_f16(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros, uint16_t* W, int N, int K) {
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            int j = k / GROUP;
            volatile float s = (float)half_bits_to_double(scales[(size_t)j * N + n]);
            volatile float z = (float)half_bits_to_double(zeros[(size_t)j * N + n]);
            volatile float d = (float)codes[(size_t)n * K + k] - z;
            volatile float p = s * d;
            _Float16 h = (_Float16)p;
            memcpy(&W[(size_t)n * K + k], &h, 2);
        }
}

/* y[m][n] = sum_k x[m][k] * ( s[j][n] * ( q[n][k] - z[j][n] ) ), fp64, k ascending. */
int slim_oracle_linear_f64(const uint16_t* x, const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                           double* y, int M, int N, int K, int threads) {
    int used = 1;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
    used = omp_get_max_threads();
#else
    (void)threads;
#endif
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                int j = k / GROUP;
                double s = half_bits_to_double(scales[(size_t)j * N + n]);
                double z = half_bits_to_double(zeros[(size_t)j * N + n]);
                double w = s * ((double)codes[(size_t)n * K + k] - z);
                acc += half_bits_to_double(x[(size_t)m * K + k]) * w;
            }
            y[(size_t)m * N + n] = acc;
        }
    return used;
}
