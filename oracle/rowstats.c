/*
 * ORACLE (test infrastructure, not product code): per-row sampling statistics on the CPU.
 *
 * For one logits row x[0..V) at a masked position i the paper's greedy estimate and confidence are
 *   r_hat_i = argmax_v P(r_i = v)           (Section 3.1, Eq. 3: greedy decoding of the clean sequence)
 *   c_i     = P(r_i = r_hat_i)              (Section 3.1, "Low-Confidence Remasking", the confidence equation)
 * with P = softmax(x) over the whole vocabulary.  So   c_i = 1 / sum_v exp(x_v - max x).
 *
 * Two values of the denominator are produced:
 *   * conf_exact : the plain definition in double precision (exp() of libm, sequential sum).
 *   * S_q        : the "canonical" fixed-point denominator (Q28) that decisions are taken on.  The paper
 *                  fixes no arithmetic; this reading makes every threshold test and every ranking
 *                  order-independent (integer addition is associative), so a parallel implementation can
 *                  reproduce the decisions bit for bit.  Steps, in fp32 IEEE arithmetic with every
 *                  operation rounded on its own (no contraction other than the written fmaf):
 *                      m   = max_v x_v ;  a = min{ v : x_v == m }
 *                      d   = x_v - m                    (exactly 0 for the maximum)
 *                      r   = fmaf(d, LOG2E, 12582912.0f)   (1.5 * 2^23: r's low mantissa bits hold n = rint(d*log2 e))
 *                      n   = r - 12582912.0f
 *                      f   = fmaf(n, -LN2, d)           (in about [-ln2/2, ln2/2])
 *                      P   = 3 + f*(C1 + f*(C2 + f*(C3 + f*C4)))   Horner, each step one fmaf; P-2 ~ e^f
 *                      e_v = ((bits(P) << 9) mod 2^32) >> (3 - n)     (0 when the shift is >= 32)
 *                      S_q = sum_v e_v          (unsigned 64-bit)
 *                  so that e_v ~ 2^28 * exp(x_v - m), truncated, the maximum contributes exactly 2^28,
 *                  and c_i ~ 2^28 / S_q.  NaN and -inf entries contribute 0.
 *   The test-suite pins S_q to conf_exact (a bound that follows from the polynomial's error and the
 *   truncation) and pins conf_exact to brute force.
 *
 * Compile:  gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC rowstats.c -o librowstats_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define SFS_ORACLE_QBITS 28

static const float kLog2e = 0x1.715476p+0f;
static const float kMagic = 12582912.0f;
static const float kLn2  = 0x1.62e430p-1f;
static const float kC1 = 0x1.fffa48p-1f;     /* e^f ~ 1 + C1 f + C2 f^2 + C3 f^3 + C4 f^4, |rel err| < 3.4e-6 on |f| <= ln2/2 */
static const float kC2 = 0x1.fff8fcp-2f;
static const float kC3 = 0x1.57f67cp-3f;
static const float kC4 = 0x1.57de66p-5f;

static inline uint32_t f32_bits(float v) { uint32_t u; memcpy(&u, &v, 4); return u; }

static inline float bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16; float f; memcpy(&f, &u, 4); return f;
}

/* one row held as fp32 values */
static void row_stats(const float *x, long V, int32_t *amax, float *vmax, uint64_t *sq, double *conf_exact)
{
    float m = -INFINITY; long a = 0;
    for (long v = 0; v < V; ++v) { if (x[v] > m) m = x[v]; }           /* NaN never wins a comparison */
    for (long v = 0; v < V; ++v) { if (x[v] == m) { a = v; break; } }   /* first maximum = lowest id (+0 == -0) */

    uint64_t S = 0;
    double   D = 0.0;
    for (long v = 0; v < V; ++v) {
        const float d = x[v] - m;
        const float r = fmaf(d, kLog2e, kMagic);
        const float n = r - kMagic;
        const float f = fmaf(n, -kLn2, d);
        float q = fmaf(f, kC4, kC3);
        q = fmaf(f, q, kC2);
        q = fmaf(f, q, kC1);
        const float P = fmaf(f, q, 3.0f);
        const uint32_t sh = 0x4B400003u - f32_bits(r);      /* = 3 - n while |d * log2 e| < 2^22 */
        const uint32_t X  = f32_bits(P) << 9;               /* drops sign+exponent: (P-2) * 2^31 */
        const uint32_t e  = (sh >= 32u) ? 0u : (X >> sh);
        S += e;
        D += exp((double)x[v] - (double)m);
    }
    *amax = (int32_t)a; *vmax = m; *sq = S; *conf_exact = 1.0 / D;
}

void sfs_oracle_rowstats_f32(const float *x, long R, long V, long ld,
                             int32_t *amax, float *vmax, uint64_t *sq, double *conf_exact)
{
    #pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < R; ++r)
        row_stats(x + r * ld, V, amax + r, vmax + r, sq + r, conf_exact + r);
}

/* bf16 logits (raw 16-bit patterns): widened exactly to fp32, then the same arithmetic */
void sfs_oracle_rowstats_bf16(const uint16_t *x, long R, long V, long ld,
                              int32_t *amax, float *vmax, uint64_t *sq, double *conf_exact)
{
    #pragma omp parallel
    {
        float *buf = (float *)__builtin_malloc(sizeof(float) * (size_t)(V > 0 ? V : 1));
        #pragma omp for schedule(dynamic, 1)
        for (long r = 0; r < R; ++r) {
            for (long v = 0; v < V; ++v) buf[v] = bf16_to_f32(x[r * ld + v]);
            row_stats(buf, V, amax + r, vmax + r, sq + r, conf_exact + r);
        }
        __builtin_free(buf);
    }
}

int sfs_oracle_qbits(void) { return SFS_ORACLE_QBITS; }
