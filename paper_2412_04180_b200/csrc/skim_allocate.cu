// Greedy bit allocation (SKIM Section 4.2, Algorithm 1) as one selection problem.
//
// Algorithm 1 raises, K times, the row whose next bit removes the most error.  Give step t of
// row i the key q(i,t) = min over u <= t of the row's u-th error reduction (a running minimum,
// so keys never increase along a row).  The sequential greedy takes exactly the first K items in
// the order (q descending, row ascending, t ascending): a row's later, larger reduction becomes
// available only once the smaller one before it has been taken, and is then taken at once.
// The kernel finds the K-th key with an 8-pass most-significant-digit radix select over the
// order-preserving 64-bit image of q, then resolves ties at the threshold by row-major rank.
#include "skim_internal.cuh"

namespace {

constexpr int AT = 1024;  // threads of the single block
constexpr int LIST_CAP = 4096;   // live keys that fit the shared-memory list of the late passes

__device__ __forceinline__ unsigned long long ordered_bits(double v)
{
    if (v == 0.0) v = 0.0;  // -0 and +0 compare equal
    const unsigned long long u = (unsigned long long)__double_as_longlong(v);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

// keys of one row: q[t] for t = 0 .. nb-2 (entries beyond stay 0); ld floats between rows of the table
__device__ __forceinline__ void row_keys(const float *err, int64_t i, int ld, int nb, unsigned long long *q)
{
    double run = 0.0;
    float prev = __ldg(err + i * ld);
#pragma unroll
    for (int t = 0; t < SKIM_MAX_NBITS - 1; ++t) {
        q[t] = 0ull;
        if (t + 1 < nb) {
            const float next = __ldg(err + i * ld + t + 1);
            const double gain = (double)prev - (double)next;
            run = (t == 0 || gain < run) ? gain : run;
            q[t] = ordered_bits(run);
            prev = next;
        }
    }
}

// Rows are dealt to threads so that a warp reads consecutive rows: warp w owns the rows
// [w * rounds * 32, (w + 1) * rounds * 32), lane l takes row j * 32 + l of that range in round j.
// CACHE_ROWS > 0: every thread keeps the keys of its (at most CACHE_ROWS) rows in registers for all
// passes; CACHE_ROWS == 0: keys are recomputed from the table in every pass.
template <int CACHE_ROWS>
__global__ void __launch_bounds__(AT) skim_allocate_kernel(const float *__restrict__ err, int64_t n, int ld, int nb,
                                                            int bmin, long long K, uint8_t *__restrict__ bits)
{
    constexpr int STEPS_MAX = SKIM_MAX_NBITS - 1;
    constexpr int NC = CACHE_ROWS > 0 ? CACHE_ROWS : 1;
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_need;
    __shared__ long long wsum[AT / 32];
    // Once few keys are still live (they share all the digits fixed so far), a pass over the table
    // also writes them to this list, and the remaining passes look at the list only.
    __shared__ unsigned long long list[LIST_CAP];
    __shared__ unsigned int s_count;             // entries of the list
    __shared__ long long s_live;                 // keys live in the coming pass
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int steps = nb - 1;

    if (K <= 0 || steps <= 0) {
        for (int64_t i = tid; i < n; i += AT) bits[i] = (uint8_t)bmin;
        return;
    }
    const int rounds = (int)((n + AT - 1) / AT);
    const int64_t row_base = (int64_t)warp * rounds * 32 + lane;

    unsigned long long cache[NC][STEPS_MAX];
    if (CACHE_ROWS > 0) {
#pragma unroll
        for (int j = 0; j < NC; ++j) {
            const int64_t i = row_base + (int64_t)j * 32;
            unsigned long long q[SKIM_MAX_NBITS] = {0ull, 0ull, 0ull, 0ull};
            if (j < rounds && i < n) row_keys(err, i, ld, nb, q);
#pragma unroll
            for (int t = 0; t < STEPS_MAX; ++t) cache[j][t] = q[t];
        }
    }
    // keys of this thread's row of round j (valid only when the row exists)
    auto keys_of = [&](int j, int64_t i, unsigned long long *q) {
        if (CACHE_ROWS > 0) {
#pragma unroll
            for (int jj = 0; jj < NC; ++jj)
                if (jj == j) {
#pragma unroll
                    for (int t = 0; t < STEPS_MAX; ++t) q[t] = cache[jj][t];
                }
        } else {
            row_keys(err, i, ld, nb, q);
        }
    };

    if (tid == 0) { s_prefix = 0ull; s_need = K; s_count = 0u; s_live = (long long)n * steps; }
    for (int d = tid; d < 256; d += AT) hist[d] = 0u;
    __syncthreads();
    bool listed = false;                         // block-uniform: the list holds every live key

    // radix select: after pass p the top 8(p+1) bits of the K-th largest key are known
    for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
        const unsigned long long prefix = s_prefix;
        if (listed) {
            const unsigned cnt = s_count;
            for (unsigned idx = tid; idx < cnt; idx += AT) {
                const unsigned long long key = list[idx];
                if ((key >> (shift + 8)) == prefix) atomicAdd(&hist[(unsigned)((key >> shift) & 0xffull)], 1u);
            }
        } else {
        const bool collect = pass >= 1 && s_live <= (long long)LIST_CAP;   // block-uniform
        // Live keys share their leading bytes, so most of a warp's keys fall into one bin: the warp
        // settles on the digit of its first live key, every lane counts its keys with that digit
        // privately, and one atomic per warp adds them all; other digits are added one by one.
        bool have_digit = false;     // warp-uniform
        unsigned d0 = 0u;
        unsigned cnt0 = 0u;
#pragma unroll (CACHE_ROWS > 0 ? NC : 1)
        for (int j = 0; j < (CACHE_ROWS > 0 ? NC : rounds); ++j) {
            if (CACHE_ROWS > 0 && j >= rounds) break;
            const int64_t i = row_base + (int64_t)j * 32;
            const bool row_ok = i < n;
            unsigned long long q[SKIM_MAX_NBITS];
            if (row_ok) keys_of(j, i, q);
            unsigned dig[STEPS_MAX];
            bool live[STEPS_MAX];
            int first = -1;
#pragma unroll
            for (int t = 0; t < STEPS_MAX; ++t) {
                const unsigned long long key = row_ok ? q[t] : 0ull;
                live[t] = row_ok && t < steps && (pass == 0 || (key >> (shift + 8)) == prefix);
                dig[t] = live[t] ? (unsigned)((key >> shift) & 0xffull) : 0u;
                if (live[t] && first < 0) first = t;
                if (collect && live[t]) {
                    const unsigned slot = atomicAdd(&s_count, 1u);
                    if (SKIM_IDX(slot, LIST_CAP, nullptr)) list[slot] = key;
                }
            }
            if (!have_digit) {
                const unsigned any = __ballot_sync(0xffffffffu, first >= 0);
                if (any) {
                    unsigned mine = 0u;
#pragma unroll
                    for (int t = 0; t < STEPS_MAX; ++t)
                        if (t == first) mine = dig[t];
                    d0 = __shfl_sync(0xffffffffu, mine, __ffs(any) - 1);
                    have_digit = true;
                }
            }
#pragma unroll
            for (int t = 0; t < STEPS_MAX; ++t) {
                if (live[t]) {
                    if (dig[t] == d0) ++cnt0;
                    else atomicAdd(&hist[dig[t]], 1u);
                }
            }
        }
        if (have_digit) {
            const unsigned total = __reduce_add_sync(0xffffffffu, cnt0);
            if (lane == 0 && total) atomicAdd(&hist[d0], total);
        }
        listed = collect;
        }
        __syncthreads();
        if (warp == 0) {
            // the digit bucket that holds the need-th largest key: suffix sums over the 256 bins
            const long long need = s_need;
            unsigned loc[8];
            long long sum = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) { loc[u] = hist[lane * 8 + u]; sum += loc[u]; }
            __syncwarp();
#pragma unroll
            for (int u = 0; u < 8; ++u) hist[lane * 8 + u] = 0u;    // ready for the next pass
            long long incl = sum;                       // bins of this lane and of all higher lanes
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const long long v = __shfl_down_sync(0xffffffffu, incl, off);
                if (lane + off < 32) incl += v;
            }
            const long long above_lane = incl - sum;    // keys in bins of higher lanes
            const bool mine = above_lane < need && need <= incl;
            const unsigned who = __ballot_sync(0xffffffffu, mine);
            if (mine || (who == 0u && lane == 0)) {
                long long above = above_lane;
                int d = 7;
                for (; d > 0; --d) {
                    if (above + (long long)loc[d] >= need) break;
                    above += loc[d];
                }
                s_need = need - above;
                s_prefix = (prefix << 8) | (unsigned long long)(lane * 8 + d);
                s_live = (long long)loc[d];
            }
        }
        __syncthreads();
    }
    const unsigned long long thr = s_prefix;   // the K-th largest key
    const long long take_eq = s_need;          // how many items equal to it are taken, in row-major order

    // items equal to the threshold are taken in row-major order: count them per warp, ...
    unsigned eq_all = 0u;
#pragma unroll (CACHE_ROWS > 0 ? NC : 1)
    for (int j = 0; j < (CACHE_ROWS > 0 ? NC : rounds); ++j) {
        if (CACHE_ROWS > 0 && j >= rounds) break;
        const int64_t i = row_base + (int64_t)j * 32;
        if (i < n) {
            unsigned long long q[SKIM_MAX_NBITS];
            keys_of(j, i, q);
#pragma unroll
            for (int t = 0; t < STEPS_MAX; ++t) eq_all += (t < steps && q[t] == thr) ? 1u : 0u;
        }
    }
    const unsigned warp_eq = __reduce_add_sync(0xffffffffu, eq_all);
    if (lane == 0) wsum[warp] = (long long)warp_eq;
    __syncthreads();
    long long carry = 0;                       // equal items in rows before this warp's current round
    for (int w = 0; w < warp; ++w) carry += wsum[w];

    // ... then rank them round by round with a warp prefix sum (rows of a round ascend with the lane)
#pragma unroll (CACHE_ROWS > 0 ? NC : 1)
    for (int j = 0; j < (CACHE_ROWS > 0 ? NC : rounds); ++j) {
        if (CACHE_ROWS > 0 && j >= rounds) break;
        const int64_t i = row_base + (int64_t)j * 32;
        const bool row_ok = i < n;
        unsigned long long q[SKIM_MAX_NBITS];
        if (row_ok) keys_of(j, i, q);
        unsigned eq = 0u;
#pragma unroll
        for (int t = 0; t < STEPS_MAX; ++t) eq += (row_ok && t < steps && q[t] == thr) ? 1u : 0u;
        unsigned inc = eq;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned v = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += v;
        }
        long long before = carry + (long long)(inc - eq);
        carry += (long long)__shfl_sync(0xffffffffu, inc, 31);
        if (row_ok) {
            int extra = 0;
#pragma unroll
            for (int t = 0; t < STEPS_MAX; ++t) {
                if (t < steps) {
                    if (q[t] > thr) {
                        ++extra;
                    } else if (q[t] == thr) {
                        if (before < take_eq) ++extra;
                        ++before;
                    }
                }
            }
            bits[i] = (uint8_t)(bmin + extra);
        }
    }
}

// Exact allocation (the dynamic programme Section 4.2 mentions as the precise but quadratic solution):
// f_i(s) = min_u f_{i-1}(s - u) + E[i-1][u] over s = bits handed out beyond b_min, smallest u on ties; one
// block walks the rows, its threads share the states; the choices are kept to walk back from s = K.
__global__ void __launch_bounds__(AT) skim_allocate_optimal_kernel(const float *__restrict__ err, int64_t n, int nb,
                                                                    int bmin, long long K, double *fa, double *fb,
                                                                    uint8_t *choice, uint8_t *__restrict__ bits,
                                                                    double *cost)
{
    const int tid = threadIdx.x;
    const double INF = __longlong_as_double(0x7ff0000000000000ll);
    for (long long s = tid; s <= K; s += AT) { fa[s] = INF; fb[s] = INF; }
    __syncthreads();
    if (tid == 0) fa[0] = 0.0;
    __syncthreads();
    double *prev = fa, *cur = fb;
    for (int64_t i = 0; i < n; ++i) {
        double e[SKIM_MAX_NBITS];
#pragma unroll
        for (int u = 0; u < SKIM_MAX_NBITS; ++u) e[u] = u < nb ? (double)__ldg(err + i * nb + u) : 0.0;
        const long long top = min(K, (long long)(i + 1) * (nb - 1));     // states beyond are unreachable (and stay infinite)
        uint8_t *ch = choice + (size_t)i * (size_t)(K + 1);
        for (long long s = tid; s <= top; s += AT) {
            double best = INF;
            int bu = 0;
#pragma unroll
            for (int u = 0; u < SKIM_MAX_NBITS; ++u) {
                if (u < nb && u <= s) {
                    const double v = prev[s - u] + e[u];
                    if (v < best) { best = v; bu = u; }
                }
            }
            cur[s] = best;
            ch[s] = (uint8_t)bu;
        }
        __syncthreads();
        double *t = prev; prev = cur; cur = t;
    }
    if (tid == 0) {
        if (cost) *cost = prev[K];
        long long s = K;
        for (int64_t i = n - 1; i >= 0; --i) {
            const int u = choice[(size_t)i * (size_t)(K + 1) + (size_t)s];
            bits[i] = (uint8_t)(bmin + u);
            s -= u;
        }
    }
}

}  // namespace

size_t skim_allocate_optimal_scratch(int64_t rows, int64_t K)
{
    const size_t f = skim_align256((size_t)(K + 1) * sizeof(double));
    return 2 * f + skim_align256((size_t)rows * (size_t)(K + 1));
}

int skim_launch_allocate_optimal(skim_ctx *ctx, const float *err, int64_t rows, const SkimBits &bits, int64_t K,
                                 void *scratch, uint8_t *out_bits, double *cost)
{
    const size_t f = skim_align256((size_t)(K + 1) * sizeof(double));
    unsigned char *p = (unsigned char *)scratch;
    skim_allocate_optimal_kernel<<<1, AT, 0, ctx->stream>>>(err, rows, bits.n_bits, bits.b_min, (long long)K, (double *)p,
                                                           (double *)(p + f), p + 2 * f, out_bits, cost);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}

int skim_launch_allocate(skim_ctx *ctx, const float *err, int64_t rows, const SkimBits &bits, int first_col, int64_t K,
                         uint8_t *out_bits)
{
    // the greedy runs on the columns first_col .. n_bits-1 of the table: every row starts at b_min + first_col
    const int ld = bits.n_bits, nb = bits.n_bits - first_col, start = bits.b_min + first_col;
    if (rows <= 4 * AT)
        skim_allocate_kernel<4><<<1, AT, 0, ctx->stream>>>(err + first_col, rows, ld, nb, start, (long long)K, out_bits);
    else
        skim_allocate_kernel<0><<<1, AT, 0, ctx->stream>>>(err + first_col, rows, ld, nb, start, (long long)K, out_bits);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
