// Row clustering: weighted 1-D K-means of every matrix row at every candidate width (SKIM
// Algorithm 3, error pre-recording loop; objective of Section 3.2, diagonal form), in two kernels
// per chunk of rows: a sort kernel (one block per row) that leaves the sorted row, its group index
// and its block prefix sums in a row record in global memory, and the Lloyd kernel (skim_lloyd.cu,
// one warp per row, thousands of rows in flight) that iterates on the records.  The split exists
// because the Lloyd iteration is a long chain of dependent small steps: inside the sort block it ran
// on one warp while two rows filled an SM's shared memory; from global memory (the hot lines stay in
// L1) every SM keeps 28 rows in flight.
//
// This file: the generic sort kernel, which handles every case -- scaled rows (32-bit keys of the
// binary32 product) and rows whose layout rules out the vectorised fp16-key kernel of
// skim_cluster16.cu -- and the host-side launcher of the whole clustering.
//
// One thread block owns one row.
//   1. load   the row's (value, importance) pairs into registers; the value is turned into an
//             order-preserving unsigned key.
//   2. sort   block-wide LSD radix sort (8-bit digits, warp-private digit counters, ballot-based
//             stable ranking), exchanging through one shared-memory buffer.  Afterwards every
//             1-D cluster is a contiguous interval of the sorted row.
//   3.        one pass over the sorted row writes its row record (skim_cluster_phases.cuh).
#include "skim_cluster_phases.cuh"

namespace {

using namespace skimk;

constexpr int RADIX_BITS = 8;
constexpr int RADIX = 1 << RADIX_BITS;

template <typename KeyT> struct Passes;
template <> struct Passes<uint32_t> { static constexpr int N = 4; };
template <> struct Passes<uint16_t> { static constexpr int N = 2; };

// Shared-memory layout, computed identically on host and device.
struct SmemLayout {
    size_t keys, gs, uni, dbase, phase, total;
};

__host__ __device__ inline SmemLayout smem_layout(int cap, int key_bytes, int nwarps)
{
    SmemLayout L;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += (b + 15) & ~(size_t)15; return o; };
    L.keys = take((size_t)cap * key_bytes);
    L.gs = take((size_t)cap * 4);
    L.uni = take((size_t)nwarps * RADIX * 4);
    L.dbase = take(RADIX * 4);
    L.phase = take(sizeof(PhaseSmem));
    L.total = off;
    return L;
}

template <typename KeyT, int THREADS, int ITEMS>
__global__ void __launch_bounds__(THREADS) skim_sort_kernel(ClusterArgs a)
{
    using K = KeyOps<KeyT>;
    constexpr int PASSES = Passes<KeyT>::N;
    constexpr int NW = THREADS / 32;
    constexpr int CAP = THREADS * ITEMS;
    extern __shared__ __align__(16) unsigned char smem[];
    const SmemLayout L = smem_layout(CAP, (int)sizeof(KeyT), NW);
    KeyT *skeys = reinterpret_cast<KeyT *>(smem + L.keys);
    float *sg = reinterpret_cast<float *>(smem + L.gs);
    uint32_t *cnt = reinterpret_cast<uint32_t *>(smem + L.uni);
    uint32_t *dbase = reinterpret_cast<uint32_t *>(smem + L.dbase);
    PhaseSmem &ps = *reinterpret_cast<PhaseSmem *>(smem + L.phase);

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int m = a.m;
    const int64_t row = a.row0 + blockIdx.x;
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
    for (int pass = 0; pass < PASSES; ++pass) {
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
            unsigned peers = 0xffffffffu;   // lanes of this warp whose item has the same digit
#pragma unroll
            for (int b = 0; b < RADIX_BITS; ++b) {
                const bool bit = (d >> b) & 1u;
                const unsigned bal = __ballot_sync(0xffffffffu, bit);
                peers &= bit ? bal : ~bal;
            }
            const uint32_t base = cnt[warp * RADIX + d];
            const unsigned rank = __popc(peers & lt_mask);
            __syncwarp();
            if (rank == 0) cnt[warp * RADIX + d] = base + __popc(peers);
            __syncwarp();
            const uint32_t pos = dbase[d] + base + rank;
            if (SKIM_IDX(pos, CAP, a.status)) {
                skeys[pos] = key[i];
                sg[pos] = val[i];
            }
        }
        __syncthreads();
        if (pass + 1 < PASSES) {
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) {
                const int e = warp * (ITEMS * 32) + i * 32 + lane;
                key[i] = skeys[e];
                val[i] = sg[e];
            }
            // the next pass re-zeroes the counters and syncs before anyone scatters again
        }
    }

    // ---------------------------------------------------------------- 3. row record for the Lloyd kernel
    if (tid == 0) { ps.misc[0] = 0; ps.misc[1] = 0; }
    __syncthreads();
    const SortedArrays<KeyT> src{skeys, sg};
    const int nd = write_row_record<KeyT, THREADS, true>(a, src, ps, 0, (int)blockIdx.x);
    if (nd <= 16) {
        collect_distinct<KeyT, THREADS>(src, m, nd, ps);
        write_distinct_values(a, nd, ps.dvals, (int)blockIdx.x);
    }
}

struct Variant {
    int cap;
    int threads;
    int key_bytes;
    void (*kernel)(ClusterArgs);
};

#define SKIM_VARIANT(KeyT, T, I) {T * I, T, (int)sizeof(KeyT), skim_sort_kernel<KeyT, T, I>}

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

// Picks the smallest variant that holds `cols` and fits shared memory.
const Variant *pick_variant(const Variant *table, int64_t cols, int max_smem, size_t *smem)
{
    for (int v = 0; v < kNumVariants; ++v) {
        if (table[v].cap < cols) continue;
        const SmemLayout L = smem_layout(table[v].cap, table[v].key_bytes, table[v].threads / 32);
        if (L.total <= (size_t)max_smem) { *smem = L.total; return &table[v]; }
    }
    return nullptr;
}

}  // namespace

int skim_cluster_max_cols(int max_smem_optin, int64_t *out)
{
    int64_t best = 0;
    for (int v = 0; v < kNumVariants; ++v) {
        size_t b;
        if (pick_variant(kVariants32, kVariants32[v].cap, max_smem_optin, &b)) best = kVariants32[v].cap;
    }
    *out = best;
    return SKIM_OK;
}

int skim_launch_cluster(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                        int64_t cols, int64_t ld, const uint8_t *row_bits, const SkimBits &bits,
                        int iters, float *centroids, uint8_t *codes, float *err, void *exact_scratch)
{
    if (rows == 0) return SKIM_OK;
    SkimWorkspace ws = skim_carve(ctx->ws, rows, cols);
    const bool scaled = ctx->scaled;
    ClusterArgs a;
    a.W = W;
    a.G = importance;
    a.rscale = scaled ? ws.rscale : nullptr;
    a.row_bits = row_bits;
    a.rows = rows;
    a.ld = ld;
    a.m = (int)cols;
    a.nb = bits.n_bits;
    a.bmin = bits.b_min;
    a.sumk = bits.sumk;
    a.iters = iters;
    a.centroids = centroids;
    a.codes = codes;
    a.err = err;
    a.status = ws.status;
    a.scratch = ws.cluster_scratch;
    a.rec_stride = 0;
    a.row0 = 0;
    a.rec_half = 0;
    a.early_exit = ctx->early_exit ? 1 : 0;
    a.iter_stats = ctx->timing ? ws.status + 1 : nullptr;

    // plan: the fp16-key sort kernel when it applies, else the generic one
    // (the exact kernel reads the full records with their g*x^2 prefixes, which only the generic kernel writes)
    bool fast = !scaled && !exact_scratch && skim_launch_sort16(ctx, a, 0, false) == SKIM_OK;
    const Variant *v = nullptr;
    size_t smem = 0;
    if (!fast) {
        v = pick_variant(scaled ? kVariants32 : kVariants16, cols, ctx->max_smem_optin, &smem);
        if (!v) return SKIM_ERR_SHAPE;
        a.rec_stride = (long long)row_record(a.m).total;
        a.rec_half = 0;
        SKIM_CUDA_OK(cudaFuncSetAttribute(v->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    if ((size_t)a.rec_stride > skim_cluster_record_bytes(cols)) return SKIM_ERR_WORKSPACE;

    for (int64_t row0 = 0; row0 < rows; row0 += SKIM_CLUSTER_CHUNK_ROWS) {
        const int64_t n = rows - row0 < SKIM_CLUSTER_CHUNK_ROWS ? rows - row0 : SKIM_CLUSTER_CHUNK_ROWS;
        a.row0 = row0;
        cudaEvent_t *tev = (ctx->timing && ctx->timing_used < SKIM_TIMING_SLOTS) ? ctx->timing_ev[ctx->timing_used] : nullptr;
        if (tev) SKIM_CUDA_OK(cudaEventRecord(tev[0], ctx->stream));
        if (fast) {
            const int rc = skim_launch_sort16(ctx, a, n, true);
            if (rc) return rc < 0 ? rc : SKIM_ERR_SHAPE;
        } else {
            v->kernel<<<(unsigned)n, v->threads, smem, ctx->stream>>>(a);
            SKIM_CUDA_OK(cudaGetLastError());
            ctx->launches += 1;
        }
        if (tev) SKIM_CUDA_OK(cudaEventRecord(tev[1], ctx->stream));
        const int rc = exact_scratch ? skim_launch_exact(ctx, a, n, exact_scratch, skim_exact_slots(ctx, rows))
                                     : skim_launch_lloyd(ctx, a, n);
        if (rc) return rc;
        if (tev) {
            SKIM_CUDA_OK(cudaEventRecord(tev[2], ctx->stream));
            ctx->timing_used += 1;
        }
    }
    return SKIM_OK;
}
