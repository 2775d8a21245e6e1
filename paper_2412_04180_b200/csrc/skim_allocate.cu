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

__device__ __forceinline__ unsigned long long ordered_bits(double v)
{
    if (v == 0.0) v = 0.0;  // -0 and +0 compare equal
    const unsigned long long u = (unsigned long long)__double_as_longlong(v);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

// keys of one row: q[t] for t = 0 .. nb-2
__device__ __forceinline__ void row_keys(const float *err, int64_t i, int nb, unsigned long long *q)
{
    double run = 0.0;
    for (int t = 0; t + 1 < nb; ++t) {
        const double gain = (double)err[i * nb + t] - (double)err[i * nb + t + 1];
        run = (t == 0 || gain < run) ? gain : run;
        q[t] = ordered_bits(run);
    }
}

__global__ void __launch_bounds__(AT) skim_allocate_kernel(const float *__restrict__ err, int64_t n, int nb,
                                                            int bmin, long long K, uint8_t *__restrict__ bits)
{
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_need;
    __shared__ long long wsum[AT / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int steps = nb - 1;

    if (K <= 0 || steps <= 0) {
        for (int64_t i = tid; i < n; i += AT) bits[i] = (uint8_t)bmin;
        return;
    }
    if (tid == 0) { s_prefix = 0ull; s_need = K; }
    __syncthreads();

    // radix select: after pass p the top 8(p+1) bits of the K-th largest key are known
    for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
        for (int d = tid; d < 256; d += AT) hist[d] = 0u;
        __syncthreads();
        const unsigned long long prefix = s_prefix;
        for (int64_t base = 0; base < n; base += AT) {
            const int64_t i = base + tid;
            unsigned long long q[SKIM_MAX_NBITS];
            if (i < n) row_keys(err, i, nb, q);
            for (int t = 0; t < steps; ++t) {
                bool live = (i < n);
                if (live && pass > 0) live = (q[t] >> (shift + 8)) == prefix;
                const unsigned d = live ? (unsigned)((q[t] >> shift) & 0xffull) : 0u;
                // keys share their leading bytes, so most lanes of a warp hold the same digit: the
                // first live lane adds the whole group at once, the others (if any) add themselves
                const unsigned livemask = __ballot_sync(0xffffffffu, live);
                if (livemask) {
                    const int leader = __ffs(livemask) - 1;
                    const unsigned d0 = __shfl_sync(0xffffffffu, d, leader);
                    const unsigned same = __ballot_sync(0xffffffffu, live && d == d0);
                    if (lane == leader) atomicAdd(&hist[d0], (unsigned)__popc(same));
                    if (live && d != d0) atomicAdd(&hist[d], 1u);
                }
            }
        }
        __syncthreads();
        if (warp == 0) {
            // the digit bucket that holds the need-th largest key: suffix sums over the 256 bins
            const long long need = s_need;
            unsigned loc[8];
            long long sum = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) { loc[u] = hist[lane * 8 + u]; sum += loc[u]; }
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
            }
        }
        __syncthreads();
    }
    const unsigned long long thr = s_prefix;   // the K-th largest key
    const long long take_eq = s_need;          // how many items equal to it are taken, in row-major order

    // rank of equal items: every thread owns a contiguous chunk of rows
    const int64_t per = (n + AT - 1) / AT;
    const int64_t r0 = min(n, (int64_t)tid * per), r1 = min(n, r0 + per);
    long long eq = 0;
    for (int64_t i = r0; i < r1; ++i) {
        unsigned long long q[SKIM_MAX_NBITS];
        row_keys(err, i, nb, q);
        for (int t = 0; t < steps; ++t) eq += (q[t] == thr) ? 1 : 0;
    }
    long long inc = eq;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const long long v = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += v;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    long long before = inc - eq;
    for (int w = 0; w < warp; ++w) before += wsum[w];

    for (int64_t i = r0; i < r1; ++i) {
        unsigned long long q[SKIM_MAX_NBITS];
        row_keys(err, i, nb, q);
        int extra = 0;
        for (int t = 0; t < steps; ++t) {
            if (q[t] > thr) {
                ++extra;
            } else if (q[t] == thr) {
                if (before < take_eq) ++extra;
                ++before;
            }
        }
        bits[i] = (uint8_t)(bmin + extra);
    }
}

}  // namespace

int skim_launch_allocate(skim_ctx *ctx, const float *err, int64_t rows, const SkimBits &bits, int64_t K,
                         uint8_t *out_bits)
{
    skim_allocate_kernel<<<1, AT, 0, ctx->stream>>>(err, rows, bits.n_bits, bits.b_min, (long long)K, out_bits);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
