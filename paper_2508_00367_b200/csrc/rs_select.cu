// Per-sample selection of the K = N - r highest-score tokens and compaction of
// the kept rows (Sec. 3.1: the reduced token set; Sec. 3.2: the r lowest-score
// tokens are removed).
//
// Selection is exact and order-stable.  fp32 scores are mapped to uint32 keys
// that sort like the floats (NaN lowest).  A 4-pass, 8-bit radix select finds
// the key of the K-th best token; tokens above it are kept, and ties at that
// key are resolved towards the lower index by a prefix count.  A block-wide
// scan of the keep flags then yields the ascending index list directly, with
// no sort.  Integer work only once the keys are formed, hence bit-exact.
#include "rs_internal.h"
#include "rs_device.cuh"
#include "rs_once.h"
#include <type_traits>

namespace rs {

namespace {

constexpr int kSelThreads = 512;

// Score of one token from the per-tile partial sums the GEMM epilogues leave (fixed summation
// order: run-to-run identical).  `enc` = number of tiles | distance << 16.  L2: sqrt of the sum of
// squares; L1: the sum; cosine: three sums per tile (u.v, u.u, v.v) -> 1 - u.v / (|u||v|).
__device__ __forceinline__ float finish_score(const float* __restrict__ p, int enc) {
    const int nparts = enc & 0xffff, dist = enc >> 16;
    if (dist == RS_DIST_COS) {
        float uv = 0.f, uu = 0.f, vv = 0.f;
        for (int j = 0; j < nparts; ++j) { uv += p[3 * j]; uu += p[3 * j + 1]; vv += p[3 * j + 2]; }
        return 1.f - uv / fmaxf(sqrtf(uu) * sqrtf(vv), 1e-12f);
    }
    float acc = 0.f;
    for (int j = 0; j < nparts; ++j) acc += p[j];
    return dist == RS_DIST_L1 ? acc : sqrtf(acc);
}
__device__ __forceinline__ int partial_stride(int enc) { return (enc & 0xffff) * ((enc >> 16) == RS_DIST_COS ? 3 : 1); }

__device__ __forceinline__ uint32_t score_key(float s) {
    if (s != s) return 0u;                 // NaN ranks below every number
    if (s == 0.f) s = 0.f;                 // -0 and +0 tie
    const uint32_t b = __float_as_uint(s);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive prefix sum over the block of one int per thread; returns the
// exclusive prefix, writes the block total to *total.  `wsum` holds >= 32 ints.
__device__ __forceinline__ int block_exclusive_scan(int v, int* wsum, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int nw = blockDim.x >> 5;
        int w = lane < nw ? wsum[lane] : 0;
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        wsum[lane] = winc - w;             // exclusive prefix of warp sums
        if (lane == 31) *total = winc;
    }
    __syncthreads();
    const int res = wsum[warp] + inc - v;
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int nparts, float* __restrict__ scores_out, int N,
              int K, int has_cls, int32_t* __restrict__ keep_idx, int32_t* __restrict__ row_map) {
    extern __shared__ uint32_t keys[];     // [N]
    __shared__ int hist[256];
    __shared__ int wsum[32];
    __shared__ int sh_bin, sh_remaining, sh_total;

    grid_dep_launch();
    grid_dep_wait();
    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    const int first = has_cls ? 1 : 0;     // token 0 is kept unconditionally when has_cls
    const int want = K - first;            // tokens to choose among indices >= first

    for (int i = tid; i < N; i += kSelThreads) {
        float s;
        if (nparts > 0) {                  // per-tile partial sums from the GEMM epilogue
            s = finish_score(scores + ((long long)b * N + i) * partial_stride(nparts), nparts);
            if (scores_out) scores_out[(long long)b * N + i] = s;
        } else {
            s = scores[(long long)b * N + i];
        }
        keys[i] = score_key(s);
    }
    __syncthreads();

    // ---- radix select: key of the want-th largest among [first, N) ----
    uint32_t prefix = 0, mask = 0;
    int remaining = want;                  // still to be taken from the candidates matching prefix
    if (want > 0) {
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            // Scores of one sample lie close together, so most keys share their upper bytes and one bin
            // takes almost every increment of a pass: lanes with the same bin add once, through one of them.
            for (int i0 = first; i0 < N; i0 += kSelThreads) {
                const int i = i0 + tid;
                uint32_t bin = 256u;                           // not a candidate of this pass
                if (i < N) {
                    const uint32_t k = keys[i];
                    if ((k & mask) == prefix) bin = (k >> shift) & 255u;
                }
                const unsigned peers = __match_any_sync(0xffffffffu, bin);
                if (bin < 256u && (tid & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
            }
            __syncthreads();
            if (tid < 32) {                // warp 0: walk the bins from the top
                int above = 0, bin = -1, rem_out = 0;
                for (int base = 224; base >= 0 && bin < 0; base -= 32) {
                    const int d = base + 31 - tid;          // lane 0 holds the highest bin
                    const int c = hist[d];
                    int inc = c;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int t = __shfl_up_sync(0xffffffffu, inc, o);
                        if (tid >= o) inc += t;
                    }
                    const int cum = above + inc;            // tokens in bins >= d
                    const bool hit = (cum >= remaining) && (cum - c < remaining);
                    const unsigned m = __ballot_sync(0xffffffffu, hit);
                    if (m) {
                        const int src = __ffs(m) - 1;
                        bin = __shfl_sync(0xffffffffu, d, src);
                        rem_out = remaining - __shfl_sync(0xffffffffu, cum - c, src);
                    }
                    above = __shfl_sync(0xffffffffu, cum, 31);
                }
                if (tid == 0) { sh_bin = bin; sh_remaining = rem_out; }
            }
            __syncthreads();
            prefix |= ((uint32_t)sh_bin) << shift;
            mask |= 255u << shift;
            remaining = sh_remaining;
            __syncthreads();
        }
    }
    const uint32_t thr = prefix;           // key of the last token that makes the cut
    // `remaining` tokens with key == thr are kept, lowest indices first.

    // ---- flags and scans over contiguous per-thread chunks ----
    const int chunk = (N + kSelThreads - 1) / kSelThreads;
    const int lo = min(tid * chunk, N), hi = min(lo + chunk, N);
    int eq_cnt = 0;
    if (want > 0)
        for (int i = max(lo, first); i < hi; ++i) eq_cnt += (keys[i] == thr);
    int eq_rank = block_exclusive_scan(eq_cnt, wsum, &sh_total);
    int kept = 0;
    for (int i = lo; i < hi; ++i) {
        bool keep;
        if (i < first) keep = true;
        else if (want <= 0) keep = false;
        else {
            const uint32_t k = keys[i];
            keep = k > thr;
            if (k == thr) { keep = eq_rank < remaining; ++eq_rank; }
        }
        keys[i] = keep ? 1u : 0u;          // the chunk is private to this thread
        kept += keep;
    }
    int pos = block_exclusive_scan(kept, wsum, &sh_total);
    int32_t* out = keep_idx + (long long)b * K;
    for (int i = lo; i < hi; ++i)
        if (keys[i]) {
            if (pos < K) {
                out[pos] = i;
                if (row_map) row_map[(long long)b * K + pos] = b * N + i;
            }
            ++pos;
        }
}

// One warp moves one kept row (16-byte pieces, all loads of a pass issued before its first store):
// to row `orow` of x_out when x_out is given, and, with LT given, LN of the row to the same row of
// ln.out.
template <int MAXV, typename LT>
__device__ __forceinline__ void copy_row(const uint4* __restrict__ src, long long orow, int row_vecs, int lane,
                                         uint4* __restrict__ x_out, const LnFuse& ln) {
    if constexpr (std::is_void<LT>::value) {
        uint4* dst = x_out + orow * row_vecs;
        float s1 = 0.f, s2 = 0.f;
        for (int base = 0; base < row_vecs; base += 32 * MAXV) {
            uint4 v[MAXV];
#pragma unroll
            for (int j = 0; j < MAXV; ++j) {
                const int iv = base + j * 32 + lane;
                if (iv < row_vecs) v[j] = __ldg(src + iv);
            }
#pragma unroll
            for (int j = 0; j < MAXV; ++j) {
                const int iv = base + j * 32 + lane;
                if (iv < row_vecs) {
                    dst[iv] = v[j];
                    if (ln.stats) {                  // bf16 rows only (the caller's business)
                        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float y0 = __uint_as_float(w[e] << 16), y1 = __uint_as_float(w[e] & 0xffff0000u);
                            s1 += y0 + y1;
                            s2 = fmaf(y0, y0, fmaf(y1, y1, s2));
                        }
                    }
                }
            }
        }
        if (ln.stats) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                s1 += __shfl_xor_sync(0xffffffffu, s1, o);
                s2 += __shfl_xor_sync(0xffffffffu, s2, o);
            }
            if (lane == 0) { ln.stats[2 * orow] = s1; ln.stats[2 * orow + 1] = s2; }
        }
    } else {
        uint4 v[MAXV];
#pragma unroll
        for (int j = 0; j < MAXV; ++j) {
            const int iv = j * 32 + lane;
            if (iv < row_vecs) v[j] = __ldg(src + iv);
        }
        if (x_out) {
            uint4* dst = x_out + orow * row_vecs;
#pragma unroll
            for (int j = 0; j < MAXV; ++j) {
                const int iv = j * 32 + lane;
                if (iv < row_vecs) dst[iv] = v[j];
            }
        }
        const int D = row_vecs * Vec16<LT>::N;
        layernorm_row<LT, LT, MAXV>(v, row_vecs, lane, ln.gamma, ln.beta, ln.eps, D, reinterpret_cast<LT*>(ln.out) + orow * D);
    }
}

// Selection by counting, and what follows it, for N <= kPruneMaxN tokens.  Token i outranks j iff
// key_i > key_j, or the keys are equal and i < j (the order the radix path realises too); its rank
// is the number of tokens that outrank it, and the K - first best-ranked candidates are kept.
// Integer work only once the keys are formed, hence bit-exact.  Two kernels: rank_kernel spreads the
// N^2 comparisons of a sample over N / P CTAs and leaves a keep flag per token and a kept count per
// slice; gather_ranked_kernel gives every kept row a warp, which finds its token from the counts and
// flags, writes the index lists and moves the row.
constexpr int kPruneMaxN = 4608;
constexpr int kRankMaxN = 2048;      // up to here the N^2 ranking spread over the grid beats the per-sample search

// Forms the N orderable keys of sample b in shared memory (finishing the scores from the GEMM's
// partial sums when they arrive that way); the scores of tokens [w0, w1) are also written out.
__device__ __forceinline__ void load_keys(const float* scores, int nparts, float* scores_out, int b, int N, int w0, int w1,
                                          uint32_t* keys) {
    for (int i = threadIdx.x; i < N; i += blockDim.x) {
        float s;
        if (nparts > 0) {
            s = finish_score(scores + ((long long)b * N + i) * partial_stride(nparts), nparts);
            if (scores_out && i >= w0 && i < w1) scores_out[(long long)b * N + i] = s;
        } else {
            s = scores[(long long)b * N + i];
        }
        keys[i] = score_key(s);
    }
}

// Keep flag of tokens [i0, i0 + P) of a sample whose keys are in shared memory: S threads (a power
// of two, a group inside a warp) per token, each counting over a strided share of the N keys.  A
// token before i outranks it on a tie, a token after it does not: two loops, one comparison each.
template <typename Put>
__device__ __forceinline__ void rank_slice(const uint32_t* keys, int N, int K, int first, int i0, int P, Put put) {
    const int nt = blockDim.x, tid = threadIdx.x, want = K - first;
    int S = 1;
    while (S < 32 && 2 * S * P <= nt) S <<= 1;
    const int sub = tid & (S - 1), per_pass = nt / S;
    for (int base = 0; base < P; base += per_pass) {
        const int t = base + tid / S, i = i0 + t;
        const bool act = t < P && i < N;
        int rank = 0;
        if (act && i >= first && want > 0) {
            const uint32_t key = keys[i];
            for (int j = first + sub; j < i; j += S) rank += keys[j] >= key;
            // first index of this thread's stride past i
            int j = i + 1 + ((sub - (i + 1 - first)) & (S - 1));
            for (; j < N; j += S) rank += keys[j] > key;
        }
        for (int o = S >> 1; o > 0; o >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
        if (act && sub == 0) put(i, (uint8_t)(i < first ? 1 : (want > 0 && rank < want) ? 1 : 0));
    }
}

// Ranking spread over the grid: CTA (g, b) ranks tokens [g P, (g+1) P) of sample b against all N
// and leaves their keep flags in global memory; N^2 / P comparisons per CTA instead of N^2.
// It also leaves the number of kept tokens of its slice in counts[b, g]: with those, whoever moves
// the rows finds the token behind an output position without scanning the sample.
// Per-sample lengths (lens, drops non-null): sample b has n_b = lens[b] tokens (clamped to 1 .. N) at
// the front of its N rows and drops r_b = drops[b] of them (clamped to 0 .. n_b - 1); the rows past
// n_b are never kept.
struct Ragged { const int32_t* lens; const int32_t* drops; int32_t* lens_out; };
__device__ __forceinline__ void sample_counts(const Ragged& rg, int b, int N, int K, int* n_b, int* k_b) {
    if (!rg.lens) { *n_b = N; *k_b = K; return; }
    const int n = min(max(__ldg(rg.lens + b), 1), N);
    const int r = min(max(__ldg(rg.drops + b), 0), n - 1);
    *n_b = n; *k_b = min(n - r, K);          // K: the row stride of the outputs, an upper bound of every count
}

__global__ void __launch_bounds__(1024)
rank_kernel(const float* __restrict__ scores, int nparts, float* __restrict__ scores_out, int N, int K, int has_cls,
            int P, uint8_t* __restrict__ flags, int32_t* __restrict__ counts, const Ragged rg, int b0) {
    __shared__ uint32_t keys[kPruneMaxN];
    __shared__ int kept_here;
    grid_dep_launch();
    grid_dep_wait();
    const int b = blockIdx.y, i0 = blockIdx.x * P;
    int n_b, k_b;
    sample_counts(rg, b0 + b, N, K, &n_b, &k_b);
    if (threadIdx.x == 0) kept_here = 0;
    load_keys(scores, nparts, scores_out, b, N, i0, i0 + P, keys);
    __syncthreads();
    uint8_t* fb = flags + (long long)b * N;
    // (the stride between samples stays N; only the first n_b keys take part)
    int mine = 0;                                        // this thread's kept tokens (at most one per pass)
    rank_slice(keys, n_b, k_b, has_cls ? 1 : 0, i0, P, [&](int i, uint8_t f) { fb[i] = f; mine += f; });
    for (int i = max(i0, n_b) + (int)threadIdx.x; i < min(i0 + P, N); i += blockDim.x) fb[i] = 0;
    mine = __reduce_add_sync(0xffffffffu, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&kept_here, mine);
    __syncthreads();
    if (threadIdx.x == 0) counts[(long long)b * gridDim.x + blockIdx.x] = kept_here;
}

// Keep flags of one sample, one CTA per sample, O(N) work per step (per-sample token counts over
// kRankMaxN tokens; with a common count the radix kernel below and the plain row kernel are faster
// there): the key t of the last token that makes the cut is found by binary search over the 32 bits
// of the key space (the largest t with at least `want` keys >= t; a block-wide count per bit, one
// counting barrier per candidate slot of a thread), tokens with a larger key are kept and the ties at
// t go to the lowest indices (a prefix count).  The same kept set as ranking every token against
// every other, without the N^2 comparisons.  Same outputs as rank_kernel: a flag per token and the
// number of kept tokens of every P-token slice in counts[b, 0 .. nsl).
__global__ void __launch_bounds__(1024)
flag_kernel(const float* __restrict__ scores, int nparts, float* __restrict__ scores_out, int N, int K, int has_cls,
            int P, int nsl, uint8_t* __restrict__ flags, int32_t* __restrict__ counts, const Ragged rg, int b0) {
    __shared__ uint32_t keys[kPruneMaxN];
    __shared__ __align__(16) uint8_t sflags[kPruneMaxN];
    __shared__ int wsum[32];
    __shared__ int sh_total;
    grid_dep_launch();
    grid_dep_wait();
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    int n_b, k_b;
    sample_counts(rg, b0 + b, N, K, &n_b, &k_b);
    const int first = has_cls ? 1 : 0, want = k_b - first;
    load_keys(scores, nparts, scores_out, b, N, 0, N, keys);
    __syncthreads();
    // this thread's candidates, strided over the sample (at most kKeysPerThread each), in registers
    constexpr int kKeysPerThread = (kPruneMaxN + 1023) / 1024;
    uint32_t kreg[kKeysPerThread];
    bool kval[kKeysPerThread];
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        const int i = first + tid + e * nt;
        kval[e] = i < n_b;
        kreg[e] = kval[e] ? keys[i] : 0u;
    }
    const int kpt = (n_b - first + nt - 1) / nt;         // candidate slots in use (the same for every thread)
    uint32_t t = 0;
    int need_eq = 0;
    if (want > 0) {
        for (int bit = 31; bit >= 0; --bit) {
            const uint32_t cand = t | (1u << bit);
            int total = 0;
#pragma unroll
            for (int e = 0; e < kKeysPerThread; ++e)
                if (e < kpt) total += __syncthreads_count(kval[e] && kreg[e] >= cand);
            if (total >= want) t = cand;
        }
        int gt = 0;
#pragma unroll
        for (int e = 0; e < kKeysPerThread; ++e)
            if (e < kpt) gt += __syncthreads_count(kval[e] && kreg[e] > t);
        need_eq = want - gt;                             // ties at t that are kept, lowest indices first
    }
    // flags over contiguous per-thread chunks, so that the ties' prefix count runs in index order
    const int chunk = (N + nt - 1) / nt;
    const int lo = min(tid * chunk, N), hi = min(lo + chunk, N);
    int eq_cnt = 0;
    if (want > 0)
        for (int i = max(lo, first); i < min(hi, n_b); ++i) eq_cnt += keys[i] == t;
    int eq_rank = block_exclusive_scan(eq_cnt, wsum, &sh_total);
    uint8_t* fb = flags + (long long)b * N;
    for (int i = lo; i < hi; ++i) {
        bool keep = false;
        if (i < first) keep = true;
        else if (i < n_b && want > 0) {
            const uint32_t k = keys[i];
            keep = k > t;
            if (k == t) { keep = eq_rank < need_eq; ++eq_rank; }
        }
        fb[i] = keep ? 1 : 0;
        sflags[i] = keep ? 1 : 0;
    }
    __syncthreads();
    // kept tokens per slice: a thread per slice adds up its P flag bytes (four at a time)
    for (int sl = tid; sl < nsl; sl += nt) {
        const int i0 = sl * P, i1 = min(i0 + P, N);
        int c = 0;
        int i = i0;
        for (; i + 4 <= i1; i += 4) c += (int)((*reinterpret_cast<const uint32_t*>(sflags + i) * 0x01010101u) >> 24);
        for (; i < i1; ++i) c += sflags[i];
        counts[(long long)b * nsl + sl] = c;
    }
}

// The rows of the kept tokens after rank_kernel or flag_kernel: one warp per output row (b, r), eight rows per
// CTA, no block-wide step.  The warp adds up the slice counts of its sample (two slices per lane,
// at most 64 slices) to find the slice that holds the r-th kept token, then the token inside the
// slice from its flags; it writes keep_idx and row_map for its row and moves the row: the dense
// copy when one is wanted and, with LT given, LN of the row for the next block.
template <int MAXV, typename LT>
__global__ void __launch_bounds__(256)
gather_ranked_kernel(const uint4* __restrict__ x, const uint8_t* __restrict__ flags, const int32_t* __restrict__ counts,
                     int nsl, int P, long long rows, int N, int K, int b0, int row_vecs, int32_t* __restrict__ keep_idx,
                     int32_t* __restrict__ row_map, uint4* __restrict__ x_out, const LnFuse ln, const Ragged rg) {
    grid_dep_launch();
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int b = (int)(row / K), r = (int)(row - (long long)b * K);
    if (rg.lens) {
        // K is the row stride of the outputs here; sample b keeps k_b <= K rows: the rest of its
        // block is zero-filled (index -1) so that whatever reads the padded buffer next sees finite rows
        int n_b, k_b;
        sample_counts(rg, b0 + b, N, K, &n_b, &k_b);
        if (r == 0 && lane == 0 && rg.lens_out) rg.lens_out[b0 + b] = k_b;
        if (r >= k_b) {
            if (lane == 0) { keep_idx[row] = -1; if (row_map) row_map[row] = -1; }
            if (x && x_out)
                for (int iv = lane; iv < row_vecs; iv += 32) x_out[row * row_vecs + iv] = make_uint4(0u, 0u, 0u, 0u);
            return;
        }
    }
    const int32_t* cb = counts + (long long)b * nsl;
    const int c0 = 2 * lane < nsl ? cb[2 * lane] : 0, c1 = 2 * lane + 1 < nsl ? cb[2 * lane + 1] : 0;
    int inc = c0 + c1;                                  // inclusive prefix over the lanes' slice pairs
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    const int before = inc - (c0 + c1);                 // kept tokens in the slices before this lane's pair
    const unsigned owner = __ballot_sync(0xffffffffu, r >= before && r < inc);
    const int src_lane = __ffs(owner) - 1;              // exactly one lane holds position r (r < K = total)
    const int pb = __shfl_sync(0xffffffffu, before, src_lane), pc0 = __shfl_sync(0xffffffffu, c0, src_lane);
    const int slice = 2 * src_lane + (r - pb >= pc0 ? 1 : 0);
    int want = r - pb - (r - pb >= pc0 ? pc0 : 0);      // position inside the slice
    const uint8_t* fb = flags + (long long)b * N + (long long)slice * P;
    const int lim = min(P, N - slice * P);
    int token = -1;
    for (int e = 0; e < lim; e += 32) {
        const bool f = e + lane < lim && fb[e + lane] != 0;
        const unsigned m = __ballot_sync(0xffffffffu, f);
        const int c = __popc(m);
        if (token < 0) {
            if (want < c) {                             // the (want+1)-th set bit of m
                unsigned mm = m;
                for (int k = 0; k < want; ++k) mm &= mm - 1;
                token = slice * P + e + (__ffs(mm) - 1);
            } else {
                want -= c;
            }
        }
    }
    if (lane == 0) {
        keep_idx[row] = token;
        if (row_map) row_map[row] = (b0 + b) * N + token;
    }
    if (x) copy_row<MAXV, LT>(x + ((long long)b * N + token) * row_vecs, row, row_vecs, lane, x_out, ln);
}

// Nothing dropped (K == N): every token is kept, in order; only the scores remain to be
// finished when they arrive as per-tile partial sums of squares.
__global__ void __launch_bounds__(256)
keep_all_kernel(const float* __restrict__ scores, int nparts, float* __restrict__ scores_out, long long T, int N,
                int32_t* __restrict__ keep_idx) {
    grid_dep_launch();
    grid_dep_wait();
    const long long t = (long long)blockIdx.x * 256 + threadIdx.x;
    if (t >= T) return;
    if (nparts > 0 && scores_out) scores_out[t] = finish_score(scores + t * partial_stride(nparts), nparts);
    keep_idx[t] = (int32_t)(t % N);
}

// x_out[b, j, :] = x[b, keep_idx[b, j], :]; one warp per kept row, 16-byte vectors,
// all loads of a row issued before the first store.
template <int MAXV, typename LT>
__global__ void __launch_bounds__(256)
gather_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ keep_idx, long long rows, int N,
              int K, int row_vecs, uint4* __restrict__ x_out, const LnFuse ln) {
    grid_dep_launch();
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const long long b = row / K;
    const int src = keep_idx[row];
    copy_row<MAXV, LT>(x + (b * N + src) * row_vecs, row, row_vecs, lane, x_out, ln);
}

// Line-wise pruning of an H x W token grid (Sec. 4, CNN variant L-W): the shift is averaged over
// every row and every column of the full grid, and the lines with the lowest averages go.  Grid
// (G, B): every CTA of sample b repeats the cheap part — one thread per line sums its line in
// fp64 in index order (the order a plain loop takes, so the averages are the same doubles on any
// machine), ranks it among its peers by counting (larger average first, lower index on a tie, NaN
// last) and the kept lines are numbered by a count over the flags — and then copies its share of
// the Hk x Wk kept positions, a warp per position.  CTA 0 of the sample writes the two index lists.
constexpr int kLineMax = 256;
constexpr int kMapMax = 8192;               // scores of one sample staged in shared memory (32 KB)

__device__ __forceinline__ bool line_outranks(double a, int ia, double b, int ib) {
    if (a != a) return (b != b) && ia < ib;
    if (b != b) return true;
    return a > b || (a == b && ia < ib);
}

template <int MAXV>
__global__ void __launch_bounds__(256)
linewise_kernel(const float* __restrict__ scores, int H, int W, int Hk, int Wk, int32_t* __restrict__ keep_rows,
                int32_t* __restrict__ keep_cols, const uint4* __restrict__ x, int row_vecs, uint4* __restrict__ x_out) {
    __shared__ double mean[2 * kLineMax];      // rows, then columns
    __shared__ int32_t kept[2 * kLineMax];
    __shared__ unsigned char flag[2 * kLineMax];
    __shared__ float smap[kMapMax];
    grid_dep_launch();
    grid_dep_wait();
    const int b = blockIdx.y;
    const float* s = scores + (long long)b * H * W;
    // a map of up to kMapMax scores is staged in shared memory first (coalesced, all threads), so
    // that the per-line loops below do not wait on global memory one element at a time
    const bool staged = H * W <= kMapMax;
    if (staged) {
        for (int i = threadIdx.x; i < H * W; i += blockDim.x) smap[i] = s[i];
        __syncthreads();
    }
    const float* sv = staged ? smap : s;
    for (int l = threadIdx.x; l < H + W; l += blockDim.x) {
        double acc = 0.0;
        if (l < H) {
            for (int w = 0; w < W; ++w) acc += (double)sv[l * W + w];
            mean[l] = acc / (double)W;
        } else {
            const int c = l - H;
            for (int h = 0; h < H; ++h) acc += (double)sv[h * W + c];
            mean[kLineMax + c] = acc / (double)H;
        }
    }
    __syncthreads();
    for (int l = threadIdx.x; l < H + W; l += blockDim.x) {
        const bool row = l < H;
        const int i = row ? l : l - H, n = row ? H : W, want = row ? Hk : Wk;
        const double* m = mean + (row ? 0 : kLineMax);
        const double mine = m[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (j != i) && line_outranks(m[j], j, mine, i);
        flag[(row ? 0 : kLineMax) + i] = rank < want;
    }
    __syncthreads();
    for (int l = threadIdx.x; l < H + W; l += blockDim.x) {
        const bool row = l < H;
        const int i = row ? l : l - H, off = row ? 0 : kLineMax;
        if (!flag[off + i]) continue;
        int pos = 0;
        for (int j = 0; j < i; ++j) pos += flag[off + j];
        kept[off + pos] = i;
        if (blockIdx.x == 0) (row ? keep_rows + (long long)b * Hk : keep_cols + (long long)b * Wk)[pos] = i;
    }
    __syncthreads();
    if (!x) return;
    const int P = Hk * Wk, G = gridDim.x, per = (P + G - 1) / G;
    const int lo = blockIdx.x * per, hi = min(lo + per, P);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const LnFuse none = {nullptr, nullptr, 0.f, nullptr, nullptr};
    auto src_of = [&](int p) {
        const int i = p / Wk, j = p - i * Wk;
        return x + (((long long)b * H + kept[i]) * W + kept[kLineMax + j]) * row_vecs;
    };
    if (row_vecs <= 32) {
        // short rows (up to 512 bytes): a warp takes 32 / rv positions side by side (rv = the row's
        // 16-byte pieces rounded up to a power of two) and four such groups per step, so that every
        // lane has four loads in flight
        int rv = 1;
        while (rv < row_vecs) rv <<= 1;
        const int side = 32 / rv, sub = lane / rv, v = lane - sub * rv, step = side * 4;
        for (int p0 = lo + warp * step; p0 < hi; p0 += nwarps * step) {
            uint4 val[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int p = p0 + u * side + sub;
                if (p < hi && v < row_vecs) val[u] = __ldg(src_of(p) + v);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int p = p0 + u * side + sub;
                if (p < hi && v < row_vecs) x_out[((long long)b * P + p) * row_vecs + v] = val[u];
            }
        }
        return;
    }
    for (int p = lo + warp; p < hi; p += nwarps)
        copy_row<MAXV, void>(src_of(p), (long long)b * P + p, row_vecs, lane, x_out, none);
}


}  // namespace

size_t select_smem_bytes(int N) { return (size_t)N * sizeof(uint32_t); }

cudaError_t select_init() {
    static PerDeviceOnce once;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    return (cudaError_t)once.run(dev, [] {
        return (int)cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
    });
}

// Scratch bytes per sample of the two-kernel path: the slice counts, then a flag per token.
static size_t prune_scratch_per_sample(int N) {
    const int P = N <= 1024 ? 64 : 128, nsl = (N + P - 1) / P;
    return (size_t)nsl * 4 + (size_t)((N + 3) / 4 * 4);
}

cudaError_t launch_select(const float* scores, int nparts, float* scores_out, int B, int N, int K,
                          int has_cls, int32_t* keep_idx, int32_t* row_map, uint8_t* flags, size_t flags_bytes,
                          int sm_count, cudaStream_t st, int* launches) {
    if (launches) *launches = 1;
    if (B == 0) return cudaSuccess;
    if (K == N) {
        const long long T = (long long)B * N;
        return launch_pdl(keep_all_kernel, dim3((unsigned)((T + 255) / 256)), dim3(256), 0, st, scores, nparts, scores_out, T, N, keep_idx);
    }
    if (prune_fusable(N, K, flags_bytes))
        return launch_prune(scores, nparts, scores_out, B, N, K, has_cls, keep_idx, row_map, RS_F32, nullptr, 0, nullptr, nullptr,
                            flags, flags_bytes, sm_count, st, launches, nullptr, nullptr, nullptr);
    return launch_pdl(select_kernel, dim3(B), dim3(kSelThreads), select_smem_bytes(N), st, scores, nparts, scores_out, N, K,
                      has_cls, keep_idx, row_map);
}

bool prune_fusable(int N, int K, size_t flags_bytes) {
    // (beyond kRankMaxN tokens the radix selection and the plain row kernel are the faster pair: 24
    // against 31 us at 4097 tokens, B = 4)
    return N <= kRankMaxN && K < N && flags_bytes >= prune_scratch_per_sample(N);
}

bool ln_fusable(rs_dtype dtype, int D) { return (size_t)D * dtype_size(dtype) / 16 <= 32 * 4; }

cudaError_t launch_prune(const float* scores, int nparts, float* scores_out, int B, int N, int K, int has_cls,
                         int32_t* keep_idx, int32_t* row_map, rs_dtype dtype, const void* x, int D, void* x_out,
                         const LnFuse* ln, uint8_t* flags, size_t flags_bytes, int sm_count, cudaStream_t st, int* launches,
                         const int32_t* seq_lens, const int32_t* drops, int32_t* lens_out) {
    const Ragged rg = {seq_lens, drops, lens_out};
    if (launches) *launches = 0;
    if (B == 0) return cudaSuccess;
    const size_t per_sample = prune_scratch_per_sample(N);
    const bool norm = ln && ln->gamma;               // else ln, if given, only asks for the row sums of the copy
    if (N > kPruneMaxN || (norm && !ln_fusable(dtype, D)) || (x && !x_out && !norm) || flags_bytes < per_sample ||
        (reinterpret_cast<uintptr_t>(flags) & 3u))
        return cudaErrorInvalidValue;
    const int row_vecs = x ? (int)((size_t)D * dtype_size(dtype) / 16) : 0;
    const size_t sz = dtype_size(dtype);
    const LnFuse none = {nullptr, nullptr, 0.f, nullptr, nullptr};
    // samples per pass: as many as the scratch holds (all of them, unless the batch is huge)
    const int Bc = (int)((flags_bytes / per_sample) < (size_t)B ? flags_bytes / per_sample : (size_t)B);
    for (int b0 = 0; b0 < B; b0 += Bc) {
        const int nb = B - b0 < Bc ? B - b0 : Bc;
        const long long t0 = (long long)b0 * N, k0 = (long long)b0 * K;
        const float* sc = scores + t0 * (nparts > 0 ? (nparts & 0xffff) * ((nparts >> 16) == RS_DIST_COS ? 3 : 1) : 1);
        float* so = scores_out ? scores_out + t0 : nullptr;
        const uint4* xs = x ? (const uint4*)((const char*)x + (size_t)t0 * D * sz) : nullptr;
        uint4* xo = x_out ? (uint4*)((char*)x_out + (size_t)k0 * D * sz) : nullptr;
        LnFuse lnc = ln ? *ln : none;
        if (norm) lnc.out = (char*)ln->out + (size_t)k0 * D * sz;
        if (ln && ln->stats) lnc.stats = ln->stats + 2 * k0;
        cudaError_t e;
        {
            // ranking: 64 tokens per CTA (4 threads each) up to 1024 tokens, else 128 (8 threads each);
            // then a warp per kept row
            const int P = N <= 1024 ? 64 : 128, nt = N <= 1024 ? 256 : 1024, nsl = (N + P - 1) / P;
            int32_t* counts = reinterpret_cast<int32_t*>(flags);
            uint8_t* fl = flags + (size_t)nb * nsl * 4;
            // (the ranking spread over the grid is the faster of the two up to kRankMaxN tokens -- 10 against
            // 14 us at 577 tokens, 17 against 20 at 1729 -- the per-sample search beyond: 31 against 57 us at 4097;
            // only batches with per-sample counts come here with more than kRankMaxN tokens)
            if (N <= kRankMaxN)
                e = launch_pdl(rank_kernel, dim3(nsl, nb), dim3(nt), 0, st, sc, nparts, so, N, K, has_cls, P, fl, counts, rg, b0);
            else
                e = launch_pdl(flag_kernel, dim3(nb), dim3(1024), 0, st, sc, nparts, so, N, K, has_cls, P, nsl, fl, counts, rg, b0);
            if (e != cudaSuccess) return e;
            const long long rows = (long long)nb * K;
            const dim3 grid((unsigned)((rows + 7) / 8)), block(256);
            int32_t* rm = row_map ? row_map + k0 : nullptr;
#define RS_GR_CASE(LT)                                                                                                  \
    launch_pdl(gather_ranked_kernel<4, LT>, grid, block, 0, st, xs, (const uint8_t*)fl, (const int32_t*)counts, nsl, P, \
               rows, N, K, b0, row_vecs, keep_idx + k0, rm, xo, lnc, rg)
            if (!norm) e = RS_GR_CASE(void);
            else if (dtype == RS_BF16) e = RS_GR_CASE(__nv_bfloat16);
            else e = RS_GR_CASE(float);
#undef RS_GR_CASE
            if (e != cudaSuccess) return e;
            if (launches) *launches += 2;
        }
    }
    return cudaSuccess;
}

cudaError_t launch_gather(rs_dtype dtype, const void* x, const int32_t* keep_idx, int B, int N, int K,
                          int D, void* x_out, const LnFuse* ln, cudaStream_t st) {
    const long long rows = (long long)B * K;
    if (rows == 0) return cudaSuccess;
    const int row_vecs = (int)((size_t)D * dtype_size(dtype) / 16);
    const unsigned grid = (unsigned)((rows + 7) / 8);
    const bool norm = ln && ln->gamma;
    if ((norm && !ln_fusable(dtype, D)) || (!x_out && !norm)) return cudaErrorInvalidValue;
    const LnFuse none = {nullptr, nullptr, 0.f, nullptr, nullptr};
#define RS_G_CASE(LT)                                                                                               \
    launch_pdl(gather_kernel<4, LT>, dim3(grid), dim3(256), 0, st, (const uint4*)x, keep_idx, rows, N, K, row_vecs, \
               (uint4*)x_out, ln ? *ln : none)
    if (!norm) return RS_G_CASE(void);
    return dtype == RS_BF16 ? RS_G_CASE(__nv_bfloat16) : RS_G_CASE(float);
#undef RS_G_CASE
}

int linewise_max_lines() { return kLineMax; }

cudaError_t launch_linewise(const float* scores, int B, int H, int W, int Hk, int Wk, int32_t* keep_rows,
                            int32_t* keep_cols, rs_dtype dtype, const void* x, int D, void* x_out, int sm_count,
                            cudaStream_t st) {
    if (B == 0) return cudaSuccess;
    const int row_vecs = x ? (int)((size_t)D * dtype_size(dtype) / 16) : 0;
    // about eight CTAs per SM in all (measured best between six and twelve), at least 16 positions
    // each; one CTA per sample for the indices alone
    int G = 1;
    if (x) {
        G = (8 * sm_count + B - 1) / B;
        const int cap = (Hk * Wk + 15) / 16;
        if (G > cap) G = cap;
        if (G < 1) G = 1;
    }
    return launch_pdl(linewise_kernel<4>, dim3(G, B), dim3(256), 0, st, scores, H, W, Hk, Wk, keep_rows, keep_cols,
                      (const uint4*)x, row_vecs, (uint4*)x_out);
}

}  // namespace rs
