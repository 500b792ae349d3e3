// WP-SGD oracle: a plain, slow, single-threaded CPU statement of what the method computes.
//
// THIS IS TEST INFRASTRUCTURE. It exists to check the CUDA library; it shares no code,
// header, table or helper with it, and nothing in the product path may call it.
//
// What it follows (Cheng, Li, Zhang, "Weighted parallel SGD for distributed
// unbalanced-workload training system"):
//   * Eq. 4      c^i(w) = (lambda/2)||w||^2 + L(x^i, y^i, w.x^i)
//   * Eq. 5      w_n = w_{n-1} - eta * d/dw c^i(w_{n-1})
//   * Algorithm 1  k nodes, node i starts from w_{i,0} and runs t - T_i steps on its own
//                  shard, then v = sum_i weight_i * w_i
//   * Eq. 6 / 8  weight_{r,i} = r^{T_i} / sum_j r^{T_j},  r = 1 - eta*lambda by default
//   * Eq. 7 / 9  the condition 2 sum_i r^{T_i} > sqrt(k) + k  (Corollary 3 / 4)
// Notation: the paper's T_i is the *delay* of node i behind the fastest node; callers here
// give step counts n_i, so t = max n_i and T_i = t - n_i.
//
// Readings where the paper is silent (each is the library's documented choice too):
//   * sample order: the n-th example of node j is row floor(u * m_j / 2^32) of its shard,
//     u the ((n-1) mod 4)-th output word of Philox4x32-10 (Salmon, Moraes, Dror, Shaw,
//     SC'11) with key = (seed low 32, seed high 32) and counter = ((n-1)/4 low 32,
//     (n-1)/4 high 32, j, 0); n is 1-based.
//   * losses (the paper names hinge/SVM only): hinge L = max(0, 1 - y z), dL/dz = -y if
//     y z < 1 else 0; logistic L = log(1 + exp(-y z)), dL/dz = -y / (1 + exp(y z));
//     squared L = (z - y)^2 / 2, dL/dz = z - y.
//   * decaying step size eta_n = eta0 / sqrt(n) (not in the paper): the weight of node j
//     generalises r^{T_j} to the product of the per-step factors (1 - eta_s lambda) over
//     the steps s = n_j+1 .. t that the node did not run; equal to Eq. 6 for constant eta.
//
// All state is fp64. Feature values are read as stored (fp32, or bf16 widened exactly).
// Pins (tests/test_oracle_*.py): pure-regulariser decay, closed-form squared-loss
// contraction, finite-difference gradients of Eq. 4, hand-computed steps, the linear-map
// form of the squared-loss chain, CSR == densified dense, lazy == literal sparse form,
// Philox known-answer vectors and an independent library generator, weight identities and
// worked values. The end-to-end v of a whole run has no value printed in the paper:
// beyond those pins, parity of v is unpinned.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

// ---- Philox4x32-10, from the published definition -------------------------------------
struct U4 { uint32_t v[4]; };

inline void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
    uint64_t p = (uint64_t)a * (uint64_t)b;
    hi = (uint32_t)(p >> 32);
    lo = (uint32_t)p;
}

U4 philox4x32_10(U4 ctr, uint32_t k0, uint32_t k1) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;  // golden ratio, sqrt(3)-1
    for (int round = 0; round < 10; ++round) {
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo(M0, ctr.v[0], hi0, lo0);
        mulhilo(M1, ctr.v[2], hi1, lo1);
        U4 nx;
        nx.v[0] = hi1 ^ ctr.v[1] ^ k0;
        nx.v[1] = lo1;
        nx.v[2] = hi0 ^ ctr.v[3] ^ k1;
        nx.v[3] = lo0;
        ctr = nx;
        k0 += W0;
        k1 += W1;
    }
    return ctr;
}

inline uint32_t sample_index(uint64_t seed, uint32_t node, int64_t n /*1-based*/, uint64_t m) {
    uint64_t q = (uint64_t)(n - 1) >> 2;
    U4 c;
    c.v[0] = (uint32_t)q;
    c.v[1] = (uint32_t)(q >> 32);
    c.v[2] = node;
    c.v[3] = 0;
    U4 o = philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
    uint32_t u = o.v[(n - 1) & 3];
    return (uint32_t)(((uint64_t)u * m) >> 32);
}

// Alternative sample order, the literal reading of Algorithm 1 ("randomly shuffle the data on machine i", then
// "get the n-th example"): one fixed pseudo-random permutation pi_j of the shard's m rows per node, cycled when
// a node runs more than m steps: the n-th example is row pi_j((n-1) mod m).
// pi_j is a keyed bijection of [0, m): a 4-round balanced Feistel network on 2w bits (2w = the even number of
// bits >= 2 that covers m-1) with cycle walking (re-encrypt until the value is < m). Round keys: the four
// output words of Philox4x32-10 at counter (0, 0, j, 1) under the seed. Round function: xor with the key,
// multiply by 0x85EBCA6B, xor-shift 13, multiply by 0xC2B2AE35, xor-shift 16 (a 32-bit integer mixer), masked
// to w bits.
inline uint32_t mix32(uint32_t x, uint32_t key) {
    uint32_t h = x ^ key;
    h *= 0x85EBCA6Bu;
    h ^= h >> 13;
    h *= 0xC2B2AE35u;
    h ^= h >> 16;
    return h;
}

inline uint32_t shuffled_index(uint64_t seed, uint32_t node, int64_t n /*1-based*/, uint64_t m) {
    if (m <= 1) return 0;
    U4 c;
    c.v[0] = 0; c.v[1] = 0; c.v[2] = node; c.v[3] = 1;
    const U4 keys = philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
    int bits = 0;
    while (((uint64_t)1 << bits) < m) ++bits;   // smallest bits with 2^bits >= m
    if (bits < 2) bits = 2;
    if (bits & 1) ++bits;
    const int w = bits / 2;
    const uint32_t mask = (w == 16) ? 0xFFFFu : (((uint32_t)1 << w) - 1u);
    uint64_t x = (uint64_t)((n - 1) % (int64_t)m);
    do {
        uint32_t L = (uint32_t)(x >> w), R = (uint32_t)x & mask;
        for (int i = 0; i < 4; ++i) {
            const uint32_t t = (L ^ mix32(R, keys.v[i])) & mask;
            L = R;
            R = t;
        }
        x = ((uint64_t)L << w) | R;
    } while (x >= m);
    return (uint32_t)x;
}

// sampling: 0 = independent uniform draws (default), 1 = shuffled order
inline uint32_t draw(int sampling, uint64_t seed, uint32_t node, int64_t n, uint64_t m) {
    return sampling == 1 ? shuffled_index(seed, node, n, m) : sample_index(seed, node, n, m);
}

inline double widen_bf16(uint16_t b) {
    uint32_t bits = (uint32_t)b << 16;
    float f;
    std::memcpy(&f, &bits, 4);
    return (double)f;
}

inline double loss_derivative(int loss, double y, double z) {
    switch (loss) {
        case 0: return (y * z < 1.0) ? -y : 0.0;           // hinge (tie y z == 1 -> 0)
        case 1: return -y / (1.0 + std::exp(y * z));        // logistic
        default: return z - y;                              // squared, L = (z-y)^2/2
    }
}

inline double step_size(double eta0, int sched, int64_t n) {
    return sched == 1 ? eta0 / std::sqrt((double)n) : eta0;
}

}  // namespace

static int g_sampling = 0;  // sample order used by the run functions (set by oracle_set_sampling)

extern "C" {

// Sample order of the run functions and of oracle_sample_indices: 0 = i.i.d. draws, 1 = shuffled order.
int oracle_set_sampling(int mode) {
    if (mode != 0 && mode != 1) return 1;
    g_sampling = mode;
    return 0;
}

// Raw generator, exposed so that tests can compare it with published vectors.
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    U4 c{{ctr[0], ctr[1], ctr[2], ctr[3]}};
    U4 o = philox4x32_10(c, key[0], key[1]);
    for (int i = 0; i < 4; ++i) out[i] = o.v[i];
}

// Row indices of steps n_begin+1 .. n_begin+count of node `node` (shard of m rows).
int oracle_sample_indices(uint64_t seed, int32_t node, int64_t m, int64_t n_begin, int64_t count,
                          uint32_t* out) {
    if (m < 1 || m > 0xFFFFFFFFLL || n_begin < 0 || count < 0 || node < 0) return 1;
    for (int64_t i = 0; i < count; ++i) out[i] = draw(g_sampling, seed, (uint32_t)node, n_begin + i + 1, (uint64_t)m);
    return 0;
}

// Algorithm 1, the per-node loop, dense rows. X is [N, ld] row-major, xtype 0 = fp32,
// 1 = bf16. W_out is [k, d] fp64: the last iterate of every node (w0 for a node with no steps).
// step_begin: the chains continue from step step_begin (so they draw examples
// step_begin+1 ...) starting at W_out's current content when resume != 0.
int oracle_run_dense(const void* X, int xtype, int64_t ld, const float* y, const int64_t* shard_off,
                     const int64_t* n_steps, int32_t k, int64_t d, float eta0_f, int sched, float lambda_f,
                     int loss, uint64_t seed, const float* w0, int64_t step_begin, int resume, double* W_out) {
    const double eta0 = (double)eta0_f, lambda = (double)lambda_f;
    std::vector<double> w((size_t)d), x((size_t)d);
    for (int32_t j = 0; j < k; ++j) {
        const int64_t m = shard_off[j + 1] - shard_off[j];
        if (n_steps[j] > 0 && m < 1) return 1;
        for (int64_t c = 0; c < d; ++c)
            w[c] = resume ? W_out[(size_t)j * d + c] : (w0 ? (double)w0[c] : 0.0);
        for (int64_t n = step_begin + 1; n <= step_begin + n_steps[j]; ++n) {
            const int64_t row = shard_off[j] + (int64_t)draw(g_sampling, seed, (uint32_t)j, n, (uint64_t)m);
            if (xtype == 1) {
                const uint16_t* xr = (const uint16_t*)X + (size_t)row * ld;
                for (int64_t c = 0; c < d; ++c) x[c] = widen_bf16(xr[c]);
            } else {
                const float* xr = (const float*)X + (size_t)row * ld;
                for (int64_t c = 0; c < d; ++c) x[c] = (double)xr[c];
            }
            double z = 0.0;
            for (int64_t c = 0; c < d; ++c) z += w[c] * x[c];
            const double g = loss_derivative(loss, (double)y[row], z);
            const double eta = step_size(eta0, sched, n);
            for (int64_t c = 0; c < d; ++c) w[c] = w[c] - eta * (lambda * w[c] + g * x[c]);
        }
        for (int64_t c = 0; c < d; ++c) W_out[(size_t)j * d + c] = w[c];
    }
    return 0;
}

// The same loop on CSR rows, written literally: every coordinate of w takes the
// regulariser term at every step (O(d) per step; for small d only).
int oracle_run_csr_literal(const int64_t* row_ptr, const int32_t* col_idx, const float* val, const float* y,
                           const int64_t* shard_off, const int64_t* n_steps, int32_t k, int64_t d,
                           float eta0_f, int sched, float lambda_f, int loss, uint64_t seed, const float* w0,
                           double* W_out) {
    const double eta0 = (double)eta0_f, lambda = (double)lambda_f;
    std::vector<double> w((size_t)d);
    for (int32_t j = 0; j < k; ++j) {
        const int64_t m = shard_off[j + 1] - shard_off[j];
        if (n_steps[j] > 0 && m < 1) return 1;
        for (int64_t c = 0; c < d; ++c) w[c] = w0 ? (double)w0[c] : 0.0;
        for (int64_t n = 1; n <= n_steps[j]; ++n) {
            const int64_t row = shard_off[j] + (int64_t)draw(g_sampling, seed, (uint32_t)j, n, (uint64_t)m);
            double z = 0.0;
            for (int64_t p = row_ptr[row]; p < row_ptr[row + 1]; ++p) z += w[col_idx[p]] * (double)val[p];
            const double g = loss_derivative(loss, (double)y[row], z);
            const double eta = step_size(eta0, sched, n);
            for (int64_t c = 0; c < d; ++c) w[c] = w[c] - eta * lambda * w[c];
            for (int64_t p = row_ptr[row]; p < row_ptr[row + 1]; ++p) w[col_idx[p]] -= eta * g * (double)val[p];
        }
        for (int64_t c = 0; c < d; ++c) W_out[(size_t)j * d + c] = w[c];
    }
    return 0;
}

// Same iterates with w = s * u: s <- s (1 - eta lambda), u_c <- u_c - (eta g / s) x_c on the
// row's nonzeros only. Algebraically identical to the literal form; used where d is large.
// With one_node >= 0 only that node is run and W_out is [d].
int oracle_run_csr_lazy(const int64_t* row_ptr, const int32_t* col_idx, const float* val, const float* y,
                        const int64_t* shard_off, const int64_t* n_steps, int32_t k, int64_t d, float eta0_f,
                        int sched, float lambda_f, int loss, uint64_t seed, const float* w0, int32_t one_node,
                        double* W_out) {
    const double eta0 = (double)eta0_f, lambda = (double)lambda_f;
    std::vector<double> u((size_t)d);
    for (int32_t j = 0; j < k; ++j) {
        if (one_node >= 0 && j != one_node) continue;
        const int64_t m = shard_off[j + 1] - shard_off[j];
        if (n_steps[j] > 0 && m < 1) return 1;
        for (int64_t c = 0; c < d; ++c) u[c] = w0 ? (double)w0[c] : 0.0;
        double s = 1.0;
        for (int64_t n = 1; n <= n_steps[j]; ++n) {
            const int64_t row = shard_off[j] + (int64_t)draw(g_sampling, seed, (uint32_t)j, n, (uint64_t)m);
            double z = 0.0;
            for (int64_t p = row_ptr[row]; p < row_ptr[row + 1]; ++p) z += u[col_idx[p]] * (double)val[p];
            z *= s;
            const double g = loss_derivative(loss, (double)y[row], z);
            const double eta = step_size(eta0, sched, n);
            s *= (1.0 - eta * lambda);
            const double coef = eta * g / s;
            if (coef != 0.0)
                for (int64_t p = row_ptr[row]; p < row_ptr[row + 1]; ++p) u[col_idx[p]] -= coef * (double)val[p];
            if (s < 1e-100) {  // fold the scale back (never reached for sensible eta*lambda)
                for (int64_t c = 0; c < d; ++c) u[c] *= s;
                s = 1.0;
            }
        }
        double* out = W_out + (one_node >= 0 ? 0 : (size_t)j * d);
        for (int64_t c = 0; c < d; ++c) out[c] = s * u[c];
    }
    return 0;
}

// Eq. 6 (r <= 0 or NaN: r = 1 - eta lambda, and for the decaying schedule the product of
// the per-step factors) and Eq. 8 (r given). cond_holds receives Eq. 7 / Eq. 9:
// 2 sum_i r^{T_i} > sqrt(k) + k. sum_rT receives sum_i r^{T_i}.
int oracle_weights(const int64_t* n_steps, int32_t k, float eta0_f, int sched, float lambda_f, double r,
                   double* weights, int* cond_holds, double* sum_rT) {
    if (k < 1) return 1;
    const double eta0 = (double)eta0_f, lambda = (double)lambda_f;
    int64_t t = 0;
    for (int32_t j = 0; j < k; ++j) {
        if (n_steps[j] < 0) return 1;
        if (n_steps[j] > t) t = n_steps[j];
    }
    const bool given = (r > 0.0);  // false for r <= 0 and for NaN
    std::vector<double> lg((size_t)k);  // log of r^{T_j}
    for (int32_t j = 0; j < k; ++j) {
        const int64_t T = t - n_steps[j];  // the paper's delay T_j
        if (given) {
            lg[j] = (double)T * std::log(r);
        } else if (sched == 0) {
            lg[j] = (double)T * std::log1p(-eta0 * lambda);
        } else {
            double a = 0.0;
            for (int64_t s = n_steps[j] + 1; s <= t; ++s) a += std::log1p(-step_size(eta0, sched, s) * lambda);
            lg[j] = a;
        }
    }
    double total = 0.0;
    for (int32_t j = 0; j < k; ++j) total += std::exp(lg[j]);
    for (int32_t j = 0; j < k; ++j) weights[j] = std::exp(lg[j]) / total;
    if (sum_rT) *sum_rT = total;
    if (cond_holds) *cond_holds = (2.0 * total > std::sqrt((double)k) + (double)k) ? 1 : 0;
    return 0;
}

// Algorithm 1, the aggregation: v = sum_j weight_j w_j, j ascending.
int oracle_combine(const double* W, const double* weights, int32_t k, int64_t d, double* v) {
    for (int64_t c = 0; c < d; ++c) {
        double a = 0.0;
        for (int32_t j = 0; j < k; ++j) a += weights[j] * W[(size_t)j * d + c];
        v[c] = a;
    }
    return 0;
}

// Objective of Eq. 3/4 on a set of dense rows: (lambda/2)||w||^2 + mean_i L(y_i, w.x_i), and the
// 0/1 error rate of sign(w.x) against y (the paper's two evaluation measures).
int oracle_objective_dense(const void* X, int xtype, int64_t ld, const float* y, int64_t n_rows, int64_t d,
                           const double* w, float lambda_f, int loss, double* objective, double* error_rate) {
    double reg = 0.0;
    for (int64_t c = 0; c < d; ++c) reg += w[c] * w[c];
    double acc = 0.0;
    int64_t wrong = 0;
    for (int64_t i = 0; i < n_rows; ++i) {
        double z = 0.0;
        if (xtype == 1) {
            const uint16_t* xr = (const uint16_t*)X + (size_t)i * ld;
            for (int64_t c = 0; c < d; ++c) z += w[c] * widen_bf16(xr[c]);
        } else {
            const float* xr = (const float*)X + (size_t)i * ld;
            for (int64_t c = 0; c < d; ++c) z += w[c] * (double)xr[c];
        }
        const double yy = (double)y[i];
        if (loss == 0) acc += std::fmax(0.0, 1.0 - yy * z);
        else if (loss == 1) acc += (yy * z > 0 ? std::log1p(std::exp(-yy * z)) : -yy * z + std::log1p(std::exp(yy * z)));
        else acc += 0.5 * (z - yy) * (z - yy);
        if ((z >= 0 ? 1.0 : -1.0) != (yy >= 0 ? 1.0 : -1.0)) ++wrong;
    }
    *objective = 0.5 * (double)lambda_f * reg + (n_rows ? acc / (double)n_rows : 0.0);
    *error_rate = n_rows ? (double)wrong / (double)n_rows : 0.0;
    return 0;
}

// The same two measures on CSR rows.
int oracle_objective_csr(const int64_t* row_ptr, const int32_t* col_idx, const float* val, const float* y,
                         int64_t n_rows, int64_t d, const double* w, float lambda_f, int loss, double* objective,
                         double* error_rate) {
    double reg = 0.0;
    for (int64_t c = 0; c < d; ++c) reg += w[c] * w[c];
    double acc = 0.0;
    int64_t wrong = 0;
    for (int64_t i = 0; i < n_rows; ++i) {
        double z = 0.0;
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) z += w[col_idx[p]] * (double)val[p];
        const double yy = (double)y[i];
        if (loss == 0) acc += std::fmax(0.0, 1.0 - yy * z);
        else if (loss == 1) acc += (yy * z > 0 ? std::log1p(std::exp(-yy * z)) : -yy * z + std::log1p(std::exp(yy * z)));
        else acc += 0.5 * (z - yy) * (z - yy);
        if ((z >= 0 ? 1.0 : -1.0) != (yy >= 0 ? 1.0 : -1.0)) ++wrong;
    }
    *objective = 0.5 * (double)lambda_f * reg + (n_rows ? acc / (double)n_rows : 0.0);
    *error_rate = n_rows ? (double)wrong / (double)n_rows : 0.0;
    return 0;
}

}  // extern "C"
