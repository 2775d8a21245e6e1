// Row clustering kernel: weighted 1-D K-means of one matrix row at every candidate width
// (SKIM Algorithm 3, error pre-recording loop; objective of Section 3.2, diagonal form).
//
// One thread block owns one row.
//   1. load   the row's (value, importance) pairs into registers; the value is turned into an
//             order-preserving unsigned key.
//   2. sort   block-wide LSD radix sort (8-bit digits, warp-private digit counters, match-based
//             stable ranking), exchanging through one shared-memory buffer.  Afterwards every
//             1-D cluster is a contiguous interval of the sorted row.
//   3. sums   binary64 prefix sums of g, g*x, g*x^2 at the granularity of small element blocks.
//   4. Lloyd  one warp, one lane per centroid of every width (2+4+8+16 = 30 lanes).  A lane owns
//             the boundary between its centroid and the next: the exact midpoint test
//             x <= (c_j + c_{j+1})/2 becomes an upper-bound search in the sorted keys, interval
//             sums are differences of prefix sums (plus the ragged ends, summed directly), the
//             new centroid is the binary64 quotient rounded to binary32.  All widths iterate in
//             lockstep; the loop ends early once no boundary moved (later iterations would
//             reproduce the same state exactly).
//   5. err    sum g (x-c)^2 per interval from the three prefix sums, in binary64.
#include "skim_internal.cuh"

namespace {

constexpr int RADIX_BITS = 8;
constexpr int RADIX = 1 << RADIX_BITS;

template <typename KeyT> struct KeyOps;

template <> struct KeyOps<uint32_t> {
    static constexpr int PASSES = 4;
    static constexpr uint32_t PAD = 0xffffffffu;
    __device__ static __forceinline__ uint32_t from_float(float x)
    {
        uint32_t u = __float_as_uint(x);
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static __forceinline__ float to_float(uint32_t k)
    {
        return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
    }
    // key of the largest representable value <= t
    __device__ static __forceinline__ uint32_t floor_key(float t) { return from_float(t); }
};

template <> struct KeyOps<uint16_t> {
    static constexpr int PASSES = 2;
    static constexpr uint16_t PAD = 0xffffu;
    __device__ static __forceinline__ uint16_t from_half_bits(uint16_t h)
    {
        return (h & 0x8000u) ? (uint16_t)~h : (uint16_t)(h | 0x8000u);
    }
    __device__ static __forceinline__ float to_float(uint16_t k)
    {
        uint16_t h = (k & 0x8000u) ? (uint16_t)(k & 0x7fffu) : (uint16_t)~k;
        return __half2float(__ushort_as_half(h));
    }
    __device__ static __forceinline__ uint16_t floor_key(float t)
    {
        uint16_t h = __half_as_ushort(__float2half_rd(t));
        if (h == 0x8000u) h = 0;
        return from_half_bits(h);
    }
};

struct ClusterArgs {
    const uint16_t *W;
    const float *G;
    const float *rscale;      // nullptr: no scale installed
    const uint8_t *row_bits;  // nullptr: every width
    int64_t rows;
    int64_t ld;
    int m;                    // cols
    int nb, bmin, sumk;
    int iters;
    int blk_shift;            // log2 of the prefix-sum block length
    float *centroids;
    uint8_t *codes;
    float *err;
    unsigned long long *status;
};

struct D3 {
    double a, b, c;
};

__device__ __forceinline__ D3 shfl_up3(D3 v, int off)
{
    D3 r;
    r.a = __shfl_up_sync(0xffffffffu, v.a, off);
    r.b = __shfl_up_sync(0xffffffffu, v.b, off);
    r.c = __shfl_up_sync(0xffffffffu, v.c, off);
    return r;
}

// Shared-memory layout, computed identically on host and device.
struct SmemLayout {
    size_t keys, gs, uni, wtot, dbase, tfs, dvals, errs, misc, total;
};

__host__ __device__ inline SmemLayout smem_layout(int cap, int key_bytes, int nwarps, int blk_shift)
{
    SmemLayout L;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += (b + 15) & ~(size_t)15; return o; };
    L.keys = take((size_t)cap * key_bytes);
    L.gs = take((size_t)cap * 4);
    size_t counters = (size_t)nwarps * RADIX * 4;
    size_t nblk = ((size_t)cap >> blk_shift) + 2;
    size_t prefix = 3 * nblk * 8;
    L.uni = take(counters > prefix ? counters : prefix);
    L.wtot = take(32 * 3 * 8);
    L.dbase = take(RADIX * 4);
    L.tfs = take(32 * 4);
    L.dvals = take(32 * 4);
    L.errs = take(32 * 8);
    L.misc = take(64);
    L.total = off;
    return L;
}

template <typename KeyT, int THREADS, int ITEMS>
__global__ void __launch_bounds__(THREADS) skim_cluster_kernel(ClusterArgs a)
{
    using K = KeyOps<KeyT>;
    constexpr int NW = THREADS / 32;
    constexpr int CAP = THREADS * ITEMS;
    extern __shared__ __align__(16) unsigned char smem[];
    const SmemLayout L = smem_layout(CAP, (int)sizeof(KeyT), NW, a.blk_shift);
    KeyT *skeys = reinterpret_cast<KeyT *>(smem + L.keys);
    float *sg = reinterpret_cast<float *>(smem + L.gs);
    uint32_t *cnt = reinterpret_cast<uint32_t *>(smem + L.uni);
    double *PB = reinterpret_cast<double *>(smem + L.uni);
    double *wtot = reinterpret_cast<double *>(smem + L.wtot);
    uint32_t *dbase = reinterpret_cast<uint32_t *>(smem + L.dbase);
    float *tfs = reinterpret_cast<float *>(smem + L.tfs);
    float *dvals = reinterpret_cast<float *>(smem + L.dvals);
    double *errs = reinterpret_cast<double *>(smem + L.errs);
    int *misc = reinterpret_cast<int *>(smem + L.misc);   // [0] distinct count, [1] slot counter

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int m = a.m;
    const int64_t row = blockIdx.x;
    const uint16_t *Wr = a.W + row * a.ld;
    const float *Gr = a.G + row * a.ld;

    // ---------------------------------------------------------------- 1. load
    KeyT key[ITEMS];
    float val[ITEMS];
    unsigned bad = 0;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const int e = warp * (ITEMS * 32) + i * 32 + lane;
        if (e < m) {
            const uint16_t h = Wr[e];
            const float g = Gr[e];
            if ((h & 0x7c00u) == 0x7c00u) bad |= 1u;
            if (!(g >= 0.0f) || g > 3.0e38f) bad |= 2u;
            if constexpr (sizeof(KeyT) == 2) {
                key[i] = KeyOps<uint16_t>::from_half_bits(h == 0x8000u ? (uint16_t)0 : h);
            } else {
                float x = __half2float(__ushort_as_half(h));
                if (a.rscale) x = __fmul_rn(x, a.rscale[e]);
                if (x == 0.0f) x = 0.0f;
                key[i] = KeyOps<uint32_t>::from_float(x);
            }
            val[i] = g;
        } else {
            key[i] = K::PAD;
            val[i] = 0.0f;
        }
    }
    if (bad) atomicOr(a.status, (unsigned long long)bad);

    // ---------------------------------------------------------------- 2. sort
    const unsigned lt_mask = (1u << lane) - 1u;
#pragma unroll 1
    for (int pass = 0; pass < K::PASSES; ++pass) {
        const int shift = pass * RADIX_BITS;
        for (int d = tid; d < NW * RADIX; d += THREADS) cnt[d] = 0;
        __syncthreads();
        // count: warp-private histogram of this digit
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const unsigned d = ((unsigned)key[i] >> shift) & (RADIX - 1);
            atomicAdd(&cnt[warp * RADIX + d], 1u);
        }
        __syncthreads();
        // scan: per digit over warps (exclusive, in place), then over digits
        for (int d = tid; d < RADIX; d += THREADS) {
            uint32_t run = 0;
            for (int w = 0; w < NW; ++w) {
                const uint32_t c = cnt[w * RADIX + d];
                cnt[w * RADIX + d] = run;
                run += c;
            }
            dbase[d] = run;
        }
        __syncthreads();
        if (warp == 0) {
            uint32_t loc[RADIX / 32];
            uint32_t s = 0;
#pragma unroll
            for (int u = 0; u < RADIX / 32; ++u) { loc[u] = dbase[lane * (RADIX / 32) + u]; s += loc[u]; }
            uint32_t inc = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += t;
            }
            uint32_t run = inc - s;
#pragma unroll
            for (int u = 0; u < RADIX / 32; ++u) { dbase[lane * (RADIX / 32) + u] = run; run += loc[u]; }
        }
        __syncthreads();
        // rank and scatter: items of one warp are taken in position order, so the pass is stable
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const unsigned d = ((unsigned)key[i] >> shift) & (RADIX - 1);
            const unsigned peers = __match_any_sync(0xffffffffu, d);
            const uint32_t base = cnt[warp * RADIX + d];
            const unsigned rank = __popc(peers & lt_mask);
            __syncwarp();
            if (rank == 0) cnt[warp * RADIX + d] = base + __popc(peers);
            __syncwarp();
            const uint32_t pos = dbase[d] + base + rank;
            skeys[pos] = key[i];
            sg[pos] = val[i];
        }
        __syncthreads();
        if (pass + 1 < K::PASSES) {
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) {
                const int e = warp * (ITEMS * 32) + i * 32 + lane;
                key[i] = skeys[e];
                val[i] = sg[e];
            }
            // the next pass re-zeroes the counters and syncs before anyone scatters again
        }
    }

    // ---------------------------------------------------------------- 3. distinct count, prefix sums
    if (tid == 0) { misc[0] = 0; misc[1] = 0; }
    __syncthreads();
    {
        int local = 0;
        for (int p = tid; p < m; p += THREADS) local += (p == 0 || skeys[p] != skeys[p - 1]) ? 1 : 0;
#pragma unroll
        for (int off = 16; off; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
        if (lane == 0 && local) atomicAdd(&misc[0], local);
    }
    const int BLK = 1 << a.blk_shift;
    const int nblk = (m + BLK - 1) >> a.blk_shift;
    double *PB0 = PB, *PB1 = PB + (nblk + 1), *PB2 = PB + 2 * (nblk + 1);
    {
        D3 carry = {0.0, 0.0, 0.0};
        for (int base = 0; base < nblk; base += THREADS) {
            const int b = base + tid;
            D3 v = {0.0, 0.0, 0.0};
            if (b < nblk) {
                const int lo = b << a.blk_shift;
                const int hi = min(m, lo + BLK);
                for (int u = lo; u < hi; ++u) {
                    const double g = (double)sg[u];
                    const double x = (double)K::to_float(skeys[u]);
                    const double gx = g * x;
                    v.a += g;
                    v.b += gx;
                    v.c = fma(gx, x, v.c);
                }
            }
            D3 inc = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const D3 t = shfl_up3(inc, off);
                if (lane >= off) { inc.a += t.a; inc.b += t.b; inc.c += t.c; }
            }
            if (lane == 31) { wtot[warp * 3 + 0] = inc.a; wtot[warp * 3 + 1] = inc.b; wtot[warp * 3 + 2] = inc.c; }
            __syncthreads();
            D3 wpre = {0.0, 0.0, 0.0}, tot = {0.0, 0.0, 0.0};
            for (int w = 0; w < NW; ++w) {
                const double t0 = wtot[w * 3 + 0], t1 = wtot[w * 3 + 1], t2 = wtot[w * 3 + 2];
                if (w < warp) { wpre.a += t0; wpre.b += t1; wpre.c += t2; }
                tot.a += t0; tot.b += t1; tot.c += t2;
            }
            if (b < nblk) {
                PB0[b] = carry.a + wpre.a + (inc.a - v.a);
                PB1[b] = carry.b + wpre.b + (inc.b - v.b);
                PB2[b] = carry.c + wpre.c + (inc.c - v.c);
            }
            carry.a += tot.a; carry.b += tot.b; carry.c += tot.c;
            __syncthreads();
        }
        if (tid == 0) { PB0[nblk] = carry.a; PB1[nblk] = carry.b; PB2[nblk] = carry.c; }
    }
    __syncthreads();
    const int nd = misc[0];   // number of distinct values in the row
    if (nd <= 16) {
        // rare: collect the distinct values (ascending) for the widths with 2^b >= nd
        for (int p = tid; p < m; p += THREADS) {
            if (p == 0 || skeys[p] != skeys[p - 1]) {
                const int slot = atomicAdd(&misc[1], 1);
                if (slot < 16) tfs[slot] = __int_as_float(p);
            }
        }
        __syncthreads();
        if (warp == 0) {
            const int p = lane < nd ? __float_as_int(tfs[lane]) : 0x7fffffff;
            int rank = 0;
            for (int u = 0; u < nd; ++u) rank += (__shfl_sync(0xffffffffu, p, u) < p) ? 1 : 0;
            __syncwarp();
            if (lane < nd) dvals[rank] = K::to_float(skeys[p]);
        }
        __syncthreads();
    }

    // ---------------------------------------------------------------- 4./5. Lloyd iterations, error
    if (warp == 0) {
        // lane -> (width index bi, centroid index j)
        int bi = 0, off = 0;
        while (bi < a.nb && lane >= off + (1 << (a.bmin + bi))) { off += 1 << (a.bmin + bi); ++bi; }
        const bool in_set = lane < a.sumk;
        const int width = a.bmin + bi;
        const int k = 1 << width;
        const int j = lane - off;
        const bool wanted = in_set && (!a.row_bits || a.row_bits[row] == width);
        const bool degenerate = wanted && (nd <= k);      // every value gets its own centroid
        const bool normal = wanted && !degenerate;
        float c = 0.0f;
        if (degenerate) c = dvals[min(j, nd - 1)];
        if (normal) c = K::to_float(skeys[(int)(((long long)(2 * j + 1) * m) / (2 * k))]);

        int Bprev = -1;
        float tf = __int_as_float(0x7f800000);            // +inf: no boundary above the last centroid
        double err_j = 0.0;
        for (int it = 0;; ++it) {
            const float c_up = __shfl_down_sync(0xffffffffu, c, 1);
            int B = m;
            if (wanted && j < k - 1) {
                tf = __double2float_rd(0.5 * ((double)c + (double)c_up));
                if (tf == 0.0f) tf = 0.0f;
                if (normal) {
                    const KeyT kt = K::floor_key(tf);
                    int lo = 0, hi = m;
                    while (lo < hi) {
                        const int mid = (lo + hi) >> 1;
                        if (skeys[mid] <= kt) lo = mid + 1; else hi = mid;
                    }
                    B = lo;
                }
            }
            const bool same = __all_sync(0xffffffffu, B == Bprev);
            const bool final = (it >= a.iters) || same;
            Bprev = B;
            D3 P = {0.0, 0.0, 0.0};
            if (normal) {
                const int blk = B >> a.blk_shift;
                P.a = PB0[blk]; P.b = PB1[blk]; P.c = PB2[blk];
                for (int u = blk << a.blk_shift; u < B; ++u) {
                    const double g = (double)sg[u];
                    const double x = (double)K::to_float(skeys[u]);
                    const double gx = g * x;
                    P.a += g;
                    P.b += gx;
                    P.c = fma(gx, x, P.c);
                }
            }
            D3 Q = shfl_up3(P, 1);
            if (j == 0) { Q.a = 0.0; Q.b = 0.0; Q.c = 0.0; }
            const double S0 = P.a - Q.a, S1 = P.b - Q.b, S2 = P.c - Q.c;
            if (final) {
                if (normal) {
                    const double cd = (double)c;
                    err_j = fmax(fma(cd, fma(cd, S0, -2.0 * S1), S2), 0.0);
                }
                break;
            }
            if (normal && S0 > 0.0) c = (float)(S1 / S0);
        }
        errs[lane] = err_j;
        tfs[lane] = (wanted && j < k - 1) ? tf : __int_as_float(0x7f800000);
        __syncwarp();
        if (wanted) {
            if (a.centroids) a.centroids[row * a.sumk + lane] = c;
            if (j == 0 && a.err) {
                double e = 0.0;
                for (int u = 0; u < k; ++u) e += errs[lane + u];
                if (a.row_bits) a.err[row] = (float)e; else a.err[row * a.nb + bi] = (float)e;
            }
        }
    }
    if (!a.codes) return;
    __syncthreads();

    // ---------------------------------------------------------------- optional: labels in column order
    {
        int only = -1;
        if (a.row_bits) only = (int)a.row_bits[row] - a.bmin;
        for (int e = tid; e < m; e += THREADS) {
            float x = __half2float(__ushort_as_half(Wr[e]));
            if (a.rscale) x = __fmul_rn(x, a.rscale[e]);
            int off = 0;
            for (int bi = 0; bi < a.nb; ++bi) {
                const int k = 1 << (a.bmin + bi);
                if (only < 0 || only == bi) {
                    int code = 0;
                    for (int u = 0; u < k - 1; ++u) code += (tfs[off + u] < x) ? 1 : 0;
                    if (only < 0) a.codes[((int64_t)bi * a.rows + row) * m + e] = (uint8_t)code;
                    else a.codes[row * (int64_t)m + e] = (uint8_t)code;
                }
                off += k;
            }
        }
    }
}

struct Variant {
    int cap;
    int threads;
    int key_bytes;
    void (*kernel)(ClusterArgs);
};

#define SKIM_VARIANT(KeyT, T, I) {T * I, T, (int)sizeof(KeyT), skim_cluster_kernel<KeyT, T, I>}

const Variant kVariants32[] = {
    SKIM_VARIANT(uint32_t, 128, 4),  SKIM_VARIANT(uint32_t, 256, 8),  SKIM_VARIANT(uint32_t, 512, 8),
    SKIM_VARIANT(uint32_t, 512, 16), SKIM_VARIANT(uint32_t, 512, 22), SKIM_VARIANT(uint32_t, 512, 32),
    SKIM_VARIANT(uint32_t, 512, 44),
};
const Variant kVariants16[] = {
    SKIM_VARIANT(uint16_t, 128, 4),  SKIM_VARIANT(uint16_t, 256, 8),  SKIM_VARIANT(uint16_t, 512, 8),
    SKIM_VARIANT(uint16_t, 512, 16), SKIM_VARIANT(uint16_t, 512, 22), SKIM_VARIANT(uint16_t, 512, 32),
    SKIM_VARIANT(uint16_t, 512, 44),
};
constexpr int kNumVariants = 7;

// Picks the smallest variant that holds `cols` and a prefix block length that fits shared memory.
const Variant *pick_variant(const Variant *table, int64_t cols, int max_smem, int *blk_shift, size_t *smem)
{
    for (int v = 0; v < kNumVariants; ++v) {
        if (table[v].cap < cols) continue;
        for (int s = 3; s <= 5; ++s) {
            const SmemLayout L = smem_layout(table[v].cap, table[v].key_bytes, table[v].threads / 32, s);
            if (L.total <= (size_t)max_smem) { *blk_shift = s; *smem = L.total; return &table[v]; }
        }
    }
    return nullptr;
}

}  // namespace

int skim_cluster_max_cols(int max_smem_optin, int64_t *out)
{
    int64_t best = 0;
    for (int v = 0; v < kNumVariants; ++v) {
        int s; size_t b;
        if (pick_variant(kVariants32, kVariants32[v].cap, max_smem_optin, &s, &b)) best = kVariants32[v].cap;
    }
    *out = best;
    return SKIM_OK;
}

int skim_launch_cluster(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                        int64_t cols, int64_t ld, const uint8_t *row_bits, const SkimBits &bits,
                        int iters, float *centroids, uint8_t *codes, float *err)
{
    if (rows == 0) return SKIM_OK;
    SkimWorkspace ws = skim_carve(ctx->ws, 0, 0);
    const bool scaled = ctx->scaled;
    int blk_shift = 3;
    size_t smem = 0;
    const Variant *v = pick_variant(scaled ? kVariants32 : kVariants16, cols, ctx->max_smem_optin, &blk_shift, &smem);
    if (!v) return SKIM_ERR_SHAPE;
    ClusterArgs a;
    a.W = W;
    a.G = importance;
    a.rscale = scaled ? skim_carve(ctx->ws, 0, ctx->scale_cols).rscale : nullptr;
    a.row_bits = row_bits;
    a.rows = rows;
    a.ld = ld;
    a.m = (int)cols;
    a.nb = bits.n_bits;
    a.bmin = bits.b_min;
    a.sumk = bits.sumk;
    a.iters = iters;
    a.blk_shift = blk_shift;
    a.centroids = centroids;
    a.codes = codes;
    a.err = err;
    a.status = ws.status;
    SKIM_CUDA_OK(cudaFuncSetAttribute(v->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    v->kernel<<<(unsigned)rows, v->threads, smem, ctx->stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
