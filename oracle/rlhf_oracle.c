/*
 * rlhf_oracle.c -- float64 CPU oracle for the token-level math of the PPO stage of RLHF.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA library is
 * checked against.  Nothing on the product path may call it; it shares no code, header, table
 * or constant with the CUDA sources.  Only the tests, the smoke check and the CPU-baseline leg
 * of the benchmark load it.
 *
 * What the paper fixes (Section 2.1, "RLHF Training"): the PPO stage keeps four models.  The
 * reference model holds the policy near its starting point, the reward model scores a whole
 * sequence, the actor is the policy being trained, the critic estimates returns.  The actor
 * generates, the four models are run in inference to build the experience, then the actor is
 * trained to raise reward while staying close to the old policy and the critic is trained on
 * the returns.  The paper prints no formula for any of it (it cites PPO, Schulman et al. 2017),
 * so every function below is the textbook definition written out in float64, and every point
 * the paper leaves open is decided in the list below.
 *
 * Pins (tests/test_oracle_*.py): closed forms, invariants, brute force, finite differences and
 * float64 torch library routines.  "Whole path vs values printed by the paper": parity
 * unpinned -- the paper prints no log-probability, reward, advantage or loss value.
 *
 * Readings where the paper is silent (Section 2.1 gives only the prose above):
 *  R1  KL penalty uses the log-probs the actor had when the experience was made (lp_old)
 *      against the reference log-probs:  kl_t = lp_old_t - lp_ref_t  (signed, unclipped).
 *  R2  reward r_t = -beta * kl_t on valid tokens; the sequence score, clipped to [-c, +c],
 *      is added at the last valid token t = len-1; nothing is added if len = 0.
 *  R3  GAE: the value after the last valid token is 0; there is no T+1-th value.
 *  R4  padded positions (t >= len) are ignored on input and produce 0 on every output.
 *  R5  no advantage whitening unless the caller asks for it (then R16).
 *  R6  both losses are token means over the whole batch: divided by N = sum_b len_b;
 *      if N = 0 both losses and every gradient are 0.
 *  R7  policy loss per token  l = max(-A*rho, -A*clip(rho, 1-eps, 1+eps)),  rho = exp(lp_new - lp_old);
 *      the gradient takes the unclipped branch when -A*rho >= -A*clip(rho) (ties included).
 *  R8  value loss per token  l = 1/2 * max((v-G)^2, (vc-G)^2),  vc = v_old + clip(v - v_old, -eps_v, +eps_v);
 *      the gradient takes the unclipped branch when (v-G)^2 >= (vc-G)^2 (ties included).
 *  R9  the two losses are returned separately, no coefficients, no entropy bonus.
 *  R10 grad_scale multiplies every gradient (it is the upstream dL).
 *  R11 a logit of -inf is a deleted vocabulary entry: it adds 0 to the partition sum and gets
 *      gradient 0.  It must not sit at the label, and a row must keep one finite logit.
 *  R12 bf16 logits are widened exactly; bf16 output rounding is round-to-nearest-even.  The same holds
 *      for IEEE binary16 (fp16) logits, the other 16-bit type the paper's model families are run in.
 *  R13 token entropy (a monitor of the policy, not a loss term: R9) is the Shannon entropy of the
 *      softmax in nats, H = -sum_v p_v log p_v; deleted entries (R11) add 0.
 *  R14 the policy-deviation monitor ("approximate KL") is the non-negative estimator
 *      mean over valid tokens of (rho - 1) - log rho,  rho = exp(lp_new - lp_old).
 *  R15 the clip fraction is the share of valid tokens whose gradient the clip switches off, i.e.
 *      whose clipped term is strictly larger than the unclipped one (the complement of R7's branch).
 *  R16 advantage whitening (optional, between GAE and the loss; off unless asked for, R5):
 *      (A - mean) / sqrt(var + eps) over the valid tokens of the whole batch, var the population
 *      variance (divided by N); padded positions give 0; N = 0 gives all zeros.
 *
 * Layout: every [B,T] array is row-major with T contiguous.  Logits are addressed as
 * base[b*stride_b + t*stride_t + v] (strides in elements), ids as ids[b*ids_stride_b + t].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef long long i64;

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* exact widening of one bf16 bit pattern (R12) */
static double bf16_to_double(uint16_t h)
{
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bf16 value, ties to even (R12); the result is returned as a
 * double.  bf16 has 8 significant bits, exponent range of float32, gradual underflow. */
double oracle_round_bf16(double x)
{
    if (isnan(x) || isinf(x) || x == 0.0) return x;
    int e;
    (void)frexp(fabs(x), &e);          /* |x| = f * 2^e with f in [0.5, 1) -> floor(log2|x|) = e-1 */
    int lg = e - 1;
    if (lg < -126) lg = -126;          /* subnormal range: fixed spacing 2^-133 */
    double ulp = ldexp(1.0, lg - 7);
    double r = nearbyint(x / ulp) * ulp;   /* default rounding mode: ties to even */
    if (fabs(r) >= ldexp(1.0, 128)) return x > 0 ? INFINITY : -INFINITY;
    return r;
}

/* exact widening of one IEEE binary16 bit pattern (R12): 1 sign, 5 exponent (bias 15), 10 fraction bits */
static double f16_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1, ex = (h >> 10) & 0x1f, fr = h & 0x3ff;
    double v;
    if (ex == 0) v = ldexp((double)fr, -24);                    /* zero and subnormals: fr * 2^-24 */
    else if (ex == 31) v = fr ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)fr / 1024.0, ex - 15);
    return sign ? -v : v;
}

double oracle_f16_to_double(uint16_t h) { return f16_to_double(h); }

/* Round a double to the nearest binary16 value, ties to even (R12); returned as a double.
 * binary16 has 11 significant bits, smallest normal 2^-14, subnormal spacing 2^-24, largest 65504. */
double oracle_round_f16(double x)
{
    if (isnan(x) || isinf(x) || x == 0.0) return x;
    int e;
    (void)frexp(fabs(x), &e);
    int lg = e - 1;
    if (lg < -14) lg = -14;
    double ulp = ldexp(1.0, lg - 10);
    double r = nearbyint(x / ulp) * ulp;
    if (fabs(r) >= 65536.0) return x > 0 ? INFINITY : -INFINITY;
    return r;
}

/* log sum_v exp(z_v), two passes: max, then sum of exp(z - max).  -inf entries add 0 (R11). */
static double row_lse(const double* z, i64 V)
{
    double mx = -INFINITY;
    for (i64 v = 0; v < V; ++v)
        if (z[v] > mx) mx = z[v];
    if (mx == -INFINITY) return -INFINITY;
    double s = 0.0;
    for (i64 v = 0; v < V; ++v)
        s += exp(z[v] - mx);
    return mx + log(s);
}

double oracle_row_lse_f64(const double* z, i64 V) { return row_lse(z, V); }

/* element type of a logits tensor: 0 = float64, 1 = bf16 bit patterns, 2 = binary16 bit patterns */
static void widen_row(const uint16_t* src, i64 V, double* dst, int dtype)
{
    if (dtype == 2) for (i64 v = 0; v < V; ++v) dst[v] = f16_to_double(src[v]);
    else for (i64 v = 0; v < V; ++v) dst[v] = bf16_to_double(src[v]);
}

/* Step 1: lp[b,t] = z[b,t,y] - log sum_v exp z[b,t,v] for t < len_b, 0 elsewhere (R4).
 * `is_bf16` selects the element type of `logits`: 0 = double, 1 = bf16 bit patterns, 2 = binary16 bit patterns.
 * Returns 0, or 1 if some id or length was out of range (that token is given lp = NaN). */
int oracle_gather_logprobs(const void* logits, int is_bf16, i64 stride_b, i64 stride_t,
                           const i64* ids, i64 ids_stride_b, const int32_t* lengths,
                           int B, int T, i64 V, double* out_lp)
{
    int bad = 0;
    i64 rows = (i64)B * T;
#pragma omp parallel
    {
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 4)
        for (i64 r = 0; r < rows; ++r) {
            int b = (int)(r / T), t = (int)(r % T);
            int len = lengths[b];
            if (len < 0 || len > T) {
#pragma omp atomic write
                bad = 1;
                out_lp[r] = 0.0;
                continue;
            }
            if (t >= len) { out_lp[r] = 0.0; continue; }
            i64 y = ids[(i64)b * ids_stride_b + t];
            if (y < 0 || y >= V) {
#pragma omp atomic write
                bad = 1;
                out_lp[r] = NAN;
                continue;
            }
            i64 off = (i64)b * stride_b + (i64)t * stride_t;
            const double* zr;
            if (is_bf16) { widen_row((const uint16_t*)logits + off, V, z, is_bf16); zr = z; }
            else zr = (const double*)logits + off;
            out_lp[r] = zr[y] - row_lse(zr, V);
        }
        free(z);
    }
    return bad;
}

/* Step 2 (R1, R2): r[b,t] = -beta*(lp_old - lp_ref) for t < len_b; the clipped score is added
 * at t = len_b - 1; 0 for t >= len_b. */
void oracle_kl_reward(const double* lp_old, const double* lp_ref, const double* score,
                      const int32_t* lengths, int B, int T, double beta, double clip,
                      double* out_r)
{
    for (int b = 0; b < B; ++b) {
        int len = lengths[b];
        for (int t = 0; t < T; ++t) {
            i64 i = (i64)b * T + t;
            if (t >= len) { out_r[i] = 0.0; continue; }
            double r = -beta * (lp_old[i] - lp_ref[i]);
            if (t == len - 1) {
                double sc = score[b];
                if (sc > clip) sc = clip;
                if (sc < -clip) sc = -clip;
                r += sc;
            }
            out_r[i] = r;
        }
    }
}

/* Step 3 (R3, R4): generalised advantage estimation, walked backwards from the last valid
 * token:  delta_t = r_t + gamma*V_{t+1} - V_t,  A_t = delta_t + gamma*lambda*A_{t+1},
 * G_t = A_t + V_t, with V_len = A_len = 0. */
void oracle_gae(const double* rewards, const double* values, const int32_t* lengths,
                int B, int T, double gamma, double lambda, double* out_adv, double* out_ret)
{
    for (int b = 0; b < B; ++b) {
        int len = lengths[b];
        double a_next = 0.0, v_next = 0.0;
        for (int t = T - 1; t >= 0; --t) {
            i64 i = (i64)b * T + t;
            if (t >= len) { out_adv[i] = 0.0; out_ret[i] = 0.0; continue; }
            double delta = rewards[i] + gamma * v_next - values[i];
            double a = delta + gamma * lambda * a_next;
            out_adv[i] = a;
            out_ret[i] = a + values[i];
            a_next = a;
            v_next = values[i];
        }
    }
}

static double clip_to(double x, double lo, double hi) { return x < lo ? lo : (x > hi ? hi : x); }

/* Step 4, the O(B*T) part (R6-R10).  Given the new log-probs of the generated tokens:
 *   loss_pg = (1/N) sum l_pg,  loss_vf = (1/N) sum l_vf  over valid tokens,
 *   out_g[b,t]  = d(grad_scale*loss_pg)/d lp_new[b,t]   (the factor in front of onehot - softmax),
 *   out_dv[b,t] = d(grad_scale*loss_vf)/d values_new[b,t]. */
void oracle_ppo_loss(const double* lp_new, const double* lp_old, const double* adv,
                     const double* values_new, const double* values_old, const double* returns,
                     const int32_t* lengths, int B, int T, double clip_eps, double value_clip,
                     double grad_scale, double* out_loss_pg, double* out_loss_vf,
                     double* out_g, double* out_dv)
{
    i64 N = 0;
    for (int b = 0; b < B; ++b) N += lengths[b];
    long double sum_pg = 0.0L, sum_vf = 0.0L;
    for (int b = 0; b < B; ++b) {
        int len = lengths[b];
        for (int t = 0; t < T; ++t) {
            i64 i = (i64)b * T + t;
            if (t >= len) { out_g[i] = 0.0; out_dv[i] = 0.0; continue; }
            double A = adv[i];
            double rho = exp(lp_new[i] - lp_old[i]);
            double unclipped = -A * rho;
            double clipped = -A * clip_to(rho, 1.0 - clip_eps, 1.0 + clip_eps);
            if (unclipped >= clipped) {
                sum_pg += unclipped;
                out_g[i] = grad_scale * unclipped / (double)N;   /* d(-A*rho)/d lp_new = -A*rho */
            } else {
                sum_pg += clipped;
                out_g[i] = 0.0;
            }
            double v = values_new[i], vo = values_old[i], G = returns[i];
            double vc = vo + clip_to(v - vo, -value_clip, value_clip);
            double e1 = (v - G) * (v - G), e2 = (vc - G) * (vc - G);
            if (e1 >= e2) {
                sum_vf += 0.5 * e1;
                out_dv[i] = grad_scale * (v - G) / (double)N;
            } else {
                sum_vf += 0.5 * e2;
                out_dv[i] = 0.0;
            }
        }
    }
    *out_loss_pg = N > 0 ? (double)(sum_pg / (long double)N) : 0.0;
    *out_loss_vf = N > 0 ? (double)(sum_vf / (long double)N) : 0.0;
}

/* Step 4, the O(V) part for a chosen list of rows (flat index b*T+t), so that no [B,T,V] float64
 * tensor ever has to exist:  dlogits[row, v] = g[row] * ([v == y] - exp(z_v - lse)).
 * Rows at padded positions, and rows with g = 0, are all zeros.  out is [n_rows, V]. */
void oracle_dlogits_rows(const void* logits, int is_bf16, i64 stride_b, i64 stride_t,
                         const i64* ids, i64 ids_stride_b, const int32_t* lengths,
                         int B, int T, i64 V, const double* g, const i64* rows, i64 n_rows,
                         double* out)
{
    (void)B;
#pragma omp parallel
    {
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 2)
        for (i64 k = 0; k < n_rows; ++k) {
            i64 r = rows[k];
            int b = (int)(r / T), t = (int)(r % T);
            double* o = out + k * V;
            if (t >= lengths[b] || g[r] == 0.0) {
                for (i64 v = 0; v < V; ++v) o[v] = 0.0;
                continue;
            }
            i64 off = (i64)b * stride_b + (i64)t * stride_t;
            const double* zr;
            if (is_bf16) { widen_row((const uint16_t*)logits + off, V, z, is_bf16); zr = z; }
            else zr = (const double*)logits + off;
            double lse = row_lse(zr, V);
            i64 y = ids[(i64)b * ids_stride_b + t];
            for (i64 v = 0; v < V; ++v) {
                double p = exp(zr[v] - lse);
                o[v] = g[r] * ((v == y ? 1.0 : 0.0) - p);
            }
        }
        free(z);
    }
}

/* Entropy of the softmax of every valid row (R13):  H = -sum_v p_v log p_v  with  p_v = exp(z_v - lse),
 * in nats; a deleted entry (z_v = -inf, p_v = 0) adds 0; 0 at padded positions.  `dtype` as `is_bf16` above. */
void oracle_token_entropy(const void* logits, int dtype, i64 stride_b, i64 stride_t,
                          const int32_t* lengths, int B, int T, i64 V, double* out_h)
{
    i64 rows = (i64)B * T;
#pragma omp parallel
    {
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 4)
        for (i64 r = 0; r < rows; ++r) {
            int b = (int)(r / T), t = (int)(r % T);
            if (t >= lengths[b]) { out_h[r] = 0.0; continue; }
            i64 off = (i64)b * stride_b + (i64)t * stride_t;
            const double* zr;
            if (dtype) { widen_row((const uint16_t*)logits + off, V, z, dtype); zr = z; }
            else zr = (const double*)logits + off;
            double lse = row_lse(zr, V);
            double h = 0.0;
            for (i64 v = 0; v < V; ++v) {
                if (zr[v] == -INFINITY) continue;
                double logp = zr[v] - lse;
                h -= exp(logp) * logp;
            }
            out_h[r] = h;
        }
        free(z);
    }
}

/* Monitors of the policy step over the valid tokens (R14, R15), from the new and old log-probs:
 *   approx_kl = (1/N) sum (rho - 1 - log rho),   clip_frac = (1/N) #{ -A*clip(rho) > -A*rho },
 * rho = exp(lp_new - lp_old).  Both 0 if N = 0. */
void oracle_ppo_stats(const double* lp_new, const double* lp_old, const double* adv,
                      const int32_t* lengths, int B, int T, double clip_eps,
                      double* out_approx_kl, double* out_clip_frac)
{
    i64 N = 0, n_clipped = 0;
    long double kl = 0.0L;
    for (int b = 0; b < B; ++b) {
        int len = lengths[b];
        N += len;
        for (int t = 0; t < len; ++t) {
            i64 i = (i64)b * T + t;
            double d = lp_new[i] - lp_old[i];
            double rho = exp(d);
            kl += (rho - 1.0) - d;
            double unclipped = -adv[i] * rho;
            double clipped = -adv[i] * clip_to(rho, 1.0 - clip_eps, 1.0 + clip_eps);
            if (clipped > unclipped) ++n_clipped;
        }
    }
    *out_approx_kl = N > 0 ? (double)(kl / (long double)N) : 0.0;
    *out_clip_frac = N > 0 ? (double)n_clipped / (double)N : 0.0;
}

/* Advantage whitening over the valid tokens of the whole batch (R16): two passes, mean then
 * population variance;  out = (A - mean) / sqrt(var + eps)  at valid positions, 0 elsewhere. */
void oracle_whiten(const double* adv, const int32_t* lengths, int B, int T, double eps, double* out)
{
    i64 N = 0;
    long double sum = 0.0L;
    for (int b = 0; b < B; ++b) {
        N += lengths[b];
        for (int t = 0; t < lengths[b]; ++t) sum += adv[(i64)b * T + t];
    }
    double mean = N > 0 ? (double)(sum / (long double)N) : 0.0;
    long double ss = 0.0L;
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < lengths[b]; ++t) {
            double d = adv[(i64)b * T + t] - mean;
            ss += d * d;
        }
    double var = N > 0 ? (double)(ss / (long double)N) : 0.0;
    double denom = sqrt(var + eps);
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < T; ++t) {
            i64 i = (i64)b * T + t;
            out[i] = (t < lengths[b] && denom > 0.0) ? (adv[i] - mean) / denom : 0.0;
        }
}
