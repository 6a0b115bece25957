// Host encoder / decoder of the lane-stream IE-BME layout (see us_host.h), the paper's own array
// layout for every other format, statistics (paper Sec. V-A storage arrays, Eq. 1) and the CTA
// schedule. Pure C++: no CUDA here.
#include <algorithm>
#include <climits>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <numeric>
#include <thread>

#include "us_host.h"

namespace us {

namespace {

int pick_threads(int threads, int64_t work_units)
{
    if (threads <= 0) threads = (int)std::thread::hardware_concurrency();
    if (threads <= 0) threads = 1;
    if ((int64_t)threads > work_units) threads = (int)std::max<int64_t>(1, work_units);
    return std::min(threads, 64);
}

template <class F>
void parallel_for(int64_t n, int threads, F&& f)
{
    threads = pick_threads(threads, n);
    if (threads == 1) {
        for (int64_t i = 0; i < n; ++i) f(i, 0);
        return;
    }
    std::vector<std::thread> pool;
    std::atomic<int64_t> next{0};
    for (int t = 0; t < threads; ++t)
        pool.emplace_back([&, t] {
            for (;;) {
                int64_t i = next.fetch_add(1);
                if (i >= n) break;
                f(i, t);
            }
        });
    for (auto& th : pool) th.join();
}

// Bitmap-aware row reordering (paper Sec. V-B, Alg. 1) in its per-strip form: within each strip
// of 16 rows, choose which rows share a union-mask row (strip rows g and g+8) so that the strip
// activates the fewest union-mask bits over the whole K extent. One choice per strip -- not per
// tile -- keeps every tile of a strip on the same output rows, so the kernel's store undoes it
// through row_order at no cost. Pair costs come from 64-bit row bitsets; the least-cost perfect
// matching is found bottom-up over all 2^16 row subsets (Eq. 5).
void pair_rows(const int8_t* W, int64_t M, int64_t K, int threads, HostMatrix* hp)
{
    HostMatrix& h = *hp;
    (void)M;
    const int64_t words = (K + 63) / 64;
    parallel_for(h.n_strips, threads, [&](int64_t rb, int) {
        std::vector<uint64_t> bits((size_t)16 * words, 0);
        for (int r = 0; r < 16; ++r) {
            const int32_t o = h.row_order[rb * 16 + r];
            if (o < 0) continue;
            const int8_t* p = W + (int64_t)o * K;
            uint64_t* b = bits.data() + (size_t)r * words;
            for (int64_t k = 0; k < K; ++k)
                if (p[k]) b[k >> 6] |= 1ull << (k & 63);
        }
        int32_t cost[16][16];
        for (int a = 0; a < 16; ++a)
            for (int b = a + 1; b < 16; ++b) {
                int64_t c = 0;
                const uint64_t *pa = bits.data() + (size_t)a * words, *pb = bits.data() + (size_t)b * words;
                for (int64_t w = 0; w < words; ++w) c += __builtin_popcountll(pa[w] | pb[w]);
                cost[a][b] = cost[b][a] = (int32_t)c;
            }
        // F[S] = least cost of pairing up the rows in S (|S| even); partner[S] = the row paired
        // with the lowest row of S in that optimum.
        std::vector<int32_t> F((size_t)1 << 16, 0);
        std::vector<int8_t> partner((size_t)1 << 16, -1);
        for (uint32_t S = 1; S < (1u << 16); ++S) {
            if (__builtin_popcount(S) & 1) continue;
            const int lo = __builtin_ctz(S);
            const uint32_t rest = S & (S - 1);
            int32_t best = INT32_MAX;
            int8_t arg = -1;
            for (uint32_t m = rest; m; m &= m - 1) {
                const int b = __builtin_ctz(m);
                const int32_t v = cost[lo][b] + F[rest & ~(1u << b)];
                if (v < best) { best = v; arg = (int8_t)b; }
            }
            F[S] = best;
            partner[S] = arg;
        }
        // Pairs come out ordered by their lower rows: the canonical order of the paper.
        int32_t old_order[16], g = 0;
        std::copy(h.row_order.begin() + rb * 16, h.row_order.begin() + rb * 16 + 16, old_order);
        for (uint32_t S = 0xFFFFu; S; ++g) {
            const int lo = __builtin_ctz(S), b = partner[S];
            h.row_order[rb * 16 + g] = old_order[lo];
            h.row_order[rb * 16 + g + 8] = old_order[b];
            S &= ~((1u << lo) | (1u << b));
        }
    });
}

}  // namespace

int32_t default_K_L(int64_t M, int64_t K, int n_sm)
{
    // Large tiles keep the per-tile padding of the lane streams and the per-tile bookkeeping small; small
    // matrices get smaller tiles so that every warp of every SM still finds work. From about four tiles of
    // 1024 columns per SM on, 1024 wins: a CTA then has no more tiles than warps, each warp decodes one tile
    // and nothing waits for a second round of copies (measured at 50 % sparsity, N = 8, K_L = 256 / 512 / 1024 /
    // 2048: 4096 x 4096 6.7 / 5.7 / 4.8 / 6.3 us, 5120 x 5120 at N = 16 10.8 / 9.1 / 8.4 / 9.8, 11008 x 4096
    // 11.9 / 10.9 / 9.0 / 8.8; 2048 x 2048 3.7 / 3.8 / 4.2 / 5.2, 1024 x 1024 3.1 / 3.4 / 3.6 / 4.5).
    const int64_t strips = (M + 15) / 16;
    if (n_sm <= 0) n_sm = 148;
    if (strips * ((K + 1023) / 1024) >= (int64_t)n_sm * 4) return 1024;
    if (strips * ((K + 511) / 512) >= (int64_t)n_sm * 4) return 512;
    return 256;
}

namespace {

// ---- the paper's own array layout, any (H_L, K_L, R_A, C_A) (Sec. V-A) ---------------------------
// Local tiles in row-block-major order; area q = a * C_A + c is the block of rows
// [a * H_L/R_A, ...) and columns [c * K_L/C_A, ...) of the tile; one union-mask bit per position
// of an area, row-major, leftmost column in the least significant bit of 64-bit words; for every
// active bit the Q values of the areas go to Q consecutive streams of P_t values each.
us_status encode_generic(const int8_t* W, int64_t M, int64_t K, const us_format& f, int threads, HostMatrix* hp)
{
    HostMatrix& h = *hp;
    const int Q = f.R_A * f.C_A, hb = f.H_L / f.R_A, kb = f.K_L / f.C_A;
    h.Mp = (M + f.H_L - 1) / f.H_L * f.H_L;
    h.Kp = (K + f.K_L - 1) / f.K_L * f.K_L;
    const int64_t tk = h.Kp / f.K_L, n_lt = (h.Mp / f.H_L) * tk;
    GenericArrays& g = h.gen;
    g.n_lt = n_lt;
    g.words_per_lt = (int64_t)hb * kb / 64;
    g.bitmaps.assign((size_t)(n_lt * g.words_per_lt), 0);
    g.offsets.assign((size_t)n_lt + 1, 0);
    std::vector<uint32_t> P((size_t)n_lt, 0);
    std::atomic<int> bad{0};
    std::atomic<int64_t> nnz{0};
    auto at = [&](int64_t r, int64_t c) -> int { return (r < M && c < K) ? W[r * K + c] : 0; };
    // pass 1: union masks and their populations
    parallel_for(n_lt, threads, [&](int64_t t, int) {
        const int64_t r0 = t / tk * f.H_L, c0 = t % tk * f.K_L;
        uint64_t* bm = g.bitmaps.data() + t * g.words_per_lt;
        uint32_t pop = 0;
        int64_t nz = 0;
        for (int i = 0; i < hb; ++i)
            for (int j = 0; j < kb; ++j) {
                bool any = false;
                for (int q = 0; q < Q; ++q) {
                    const int v = at(r0 + (q / f.C_A) * hb + i, c0 + (q % f.C_A) * kb + j);
                    if (v < -8 || v > 7) bad.store(1);
                    if (v) { any = true; ++nz; }
                }
                if (any) {
                    const int64_t bit = (int64_t)i * kb + j;
                    bm[bit >> 6] |= 1ull << (bit & 63);
                    ++pop;
                }
            }
        P[t] = pop;
        nnz += nz;
    });
    if (bad.load()) return US_ERR_VALUE_RANGE;
    uint64_t o = 0;
    for (int64_t t = 0; t < n_lt; ++t) {
        g.offsets[t] = (uint32_t)o;
        o += (uint64_t)Q * P[t];
        if (o > 0xFFFFFFFFull) return US_ERR_ALLOC;
    }
    g.offsets[n_lt] = (uint32_t)o;
    g.values.assign((size_t)((o + 1) / 2), 0);
    // pass 2: the value streams (two tiles never share a byte only when their offsets are even;
    // an odd total would make neighbours share one, so this pass runs tile after tile)
    for (int64_t t = 0; t < n_lt; ++t) {
        const int64_t r0 = t / tk * f.H_L, c0 = t % tk * f.K_L;
        const uint64_t* bm = g.bitmaps.data() + t * g.words_per_lt;
        uint64_t rank = 0;
        for (int64_t bit = 0; bit < (int64_t)hb * kb; ++bit) {
            if (!((bm[bit >> 6] >> (bit & 63)) & 1)) continue;
            const int i = (int)(bit / kb), j = (int)(bit % kb);
            for (int q = 0; q < Q; ++q) {
                const uint64_t idx = g.offsets[t] + (uint64_t)q * P[t] + rank;
                const uint8_t nib = (uint8_t)at(r0 + (q / f.C_A) * hb + i, c0 + (q % f.C_A) * kb + j) & 0xF;
                g.values[idx >> 1] |= (uint8_t)(nib << (4 * (idx & 1)));
            }
            ++rank;
        }
        h.sum_P += P[t];
    }
    h.nnz = nnz.load();
    h.n_strips = h.Mp / f.H_L;
    h.n_segs = tk;
    return US_OK;
}

void decode_generic(const HostMatrix& h, int8_t* W_out)
{
    const us_format& f = h.fmt;
    const GenericArrays& g = h.gen;
    const int Q = f.R_A * f.C_A, hb = f.H_L / f.R_A, kb = f.K_L / f.C_A;
    const int64_t tk = h.Kp / f.K_L;
    for (int64_t t = 0; t < g.n_lt; ++t) {
        const int64_t r0 = t / tk * f.H_L, c0 = t % tk * f.K_L;
        const uint64_t* bm = g.bitmaps.data() + t * g.words_per_lt;
        const uint64_t P = (g.offsets[t + 1] - g.offsets[t]) / (uint64_t)Q;
        uint64_t rank = 0;
        for (int64_t bit = 0; bit < (int64_t)hb * kb; ++bit) {
            if (!((bm[bit >> 6] >> (bit & 63)) & 1)) continue;
            const int i = (int)(bit / kb), j = (int)(bit % kb);
            for (int q = 0; q < Q; ++q) {
                const uint64_t idx = g.offsets[t] + (uint64_t)q * P + rank;
                const int nib = (g.values[idx >> 1] >> (4 * (idx & 1))) & 0xF;
                const int64_t r = r0 + (q / f.C_A) * hb + i, c = c0 + (q % f.C_A) * kb + j;
                if (r < h.M && c < h.K) W_out[r * h.K + c] = (int8_t)(nib >= 8 ? nib - 16 : nib);
            }
            ++rank;
        }
    }
}

}  // namespace

us_status encode_host(const int8_t* W, int64_t M, int64_t K, const uint16_t* w_scale,
                      const us_format& fmt, uint32_t flags, int threads, HostMatrix* out)
{
    if (!W || !out || M <= 0 || K <= 0) return US_ERR_INVALID_ARG;
    if (fmt.H_L <= 0 || fmt.K_L <= 0 || fmt.R_A <= 0 || fmt.C_A <= 0) return US_ERR_SHAPE;
    if (fmt.H_L % fmt.R_A || fmt.K_L % fmt.C_A) return US_ERR_SHAPE;
    if (((int64_t)(fmt.H_L / fmt.R_A) * (fmt.K_L / fmt.C_A)) % 64) return US_ERR_SHAPE;

    HostMatrix& h = *out;
    h = HostMatrix();
    h.M = M; h.K = K; h.fmt = fmt;
    h.kernel_layout = fmt.H_L == 16 && fmt.R_A == 2 && fmt.K_L <= 8192 &&
                      ((fmt.C_A == 1 && fmt.K_L % 128 == 0) || (fmt.C_A == 2 && fmt.K_L % 256 == 0));
    h.w2 = (flags & US_ENCODE_W2) != 0;
    // INT2 weights: only in the folded kernel layout, where a mask bit's four values fill one byte
    if (h.w2 && !(h.kernel_layout && fmt.C_A == 2)) { h = HostMatrix(); return US_ERR_UNSUPPORTED; }
    if (h.w2 && (flags & US_ENCODE_PAIR_ROWS)) { h = HostMatrix(); return US_ERR_UNSUPPORTED; }
    if (!h.kernel_layout) {
        // a valid IE-BME format without a kernel: the paper's arrays, for statistics and decoding
        if (!(flags & US_ENCODE_HOST_ONLY)) return US_ERR_UNSUPPORTED;
        if (flags & (US_ENCODE_SORT_ROWS | US_ENCODE_PAIR_ROWS)) return US_ERR_UNSUPPORTED;
        if ((int64_t)fmt.H_L * fmt.K_L > (1 << 24)) return US_ERR_UNSUPPORTED;
        if (w_scale) h.w_scale.assign(w_scale, w_scale + M);
        us_status st = encode_generic(W, M, K, fmt, threads, &h);
        if (st != US_OK) h = HostMatrix();
        return st;
    }
    h.Mp = (M + 15) / 16 * 16;
    h.Kp = (K + fmt.K_L - 1) / fmt.K_L * fmt.K_L;
    h.nkb = fmt.K_L / 32;
    h.mask_rows = h.nkb / (4 * fmt.C_A);
    // the pairing cost below is written for one column area
    if (fmt.C_A == 2 && (flags & US_ENCODE_PAIR_ROWS)) { h = HostMatrix(); return US_ERR_UNSUPPORTED; }
    h.n_strips = h.Mp / 16;
    h.n_segs = h.Kp / fmt.K_L;
    h.n_items = h.n_strips * h.n_segs;
    if (w_scale) h.w_scale.assign(w_scale, w_scale + M);

    // ---- row order -----------------------------------------------------------------------
    h.row_order.assign(h.Mp, -1);
    std::atomic<int> bad{0};
    if (flags & US_ENCODE_SORT_ROWS) {
        std::vector<int64_t> cnt(M, 0);
        parallel_for(M, threads, [&](int64_t r, int) {
            const int8_t* p = W + r * K;
            int64_t c = 0;
            for (int64_t k = 0; k < K; ++k) c += p[k] != 0;
            cnt[r] = c;
        });
        std::vector<int32_t> idx(M);
        std::iota(idx.begin(), idx.end(), 0);
        std::stable_sort(idx.begin(), idx.end(), [&](int32_t a, int32_t b) { return cnt[a] < cnt[b]; });
        std::copy(idx.begin(), idx.end(), h.row_order.begin());
    } else {
        std::iota(h.row_order.begin(), h.row_order.begin() + M, 0);
    }

    if (flags & US_ENCODE_PAIR_ROWS) pair_rows(W, M, K, threads, &h);

    // ---- build every tile blob (parallel over strips) ------------------------------------
    const int K_L = fmt.K_L, CA = fmt.C_A, nkb = h.nkb / CA, mask_rows = h.mask_rows;   // nkb: mask bytes per lane
    const bool w2 = h.w2;
    const int vmin = w2 ? -2 : -8, vmax = w2 ? 1 : 7;
    const int SR = w2 ? 1 : CA;   // payload streams per lane (INT2: the two column areas share a byte)
    const int K_B = K_L / CA;                                                            // columns per column area
    const int64_t mask_bytes = (int64_t)mask_rows * 128;
    std::vector<std::vector<uint8_t>> blobs(h.n_items);
    std::atomic<int64_t> nnz{0}, sum_P{0};

    parallel_for(h.n_strips, threads, [&](int64_t rb, int) {
        const int8_t* rows[16];
        for (int r = 0; r < 16; ++r) {
            int32_t o = h.row_order[rb * 16 + r];
            rows[r] = o < 0 ? nullptr : W + (int64_t)o * K;
        }
        std::vector<uint8_t> stream((size_t)32 * nkb * 8);  // lane-major payload bytes (column area 0)
        std::vector<uint8_t> stream2(CA == 2 ? (size_t)32 * nkb * 8 : 0);   // column area 1
        std::vector<uint8_t> mask((size_t)32 * nkb);        // lane-major mask bytes
        int len[32];
        int64_t my_nnz = 0, my_P = 0;
        for (int64_t sg = 0; sg < h.n_segs; ++sg) {
            const int64_t k0 = sg * K_L;
            std::fill(mask.begin(), mask.end(), 0);
            std::fill(len, len + 32, 0);
            for (int g = 0; g < 8; ++g) {
                const int8_t* pa = rows[g];
                const int8_t* pb = rows[g + 8];
                // kk = column within the column area; with C_A = 2 one mask bit covers columns kk and
                // kk + K_B of the tile (rows g and g + 8 of each), and the two columns' bytes go to two
                // streams of equal length
                for (int kk = 0; kk < K_B; ++kk) {
                    int v[2][2];   // [column area][row half]
                    int any = 0;
                    for (int ca = 0; ca < CA; ++ca) {
                        const int64_t k = k0 + kk + (int64_t)ca * K_B;
                        v[ca][0] = (pa && k < K) ? pa[k] : 0;
                        v[ca][1] = (pb && k < K) ? pb[k] : 0;
                        any |= v[ca][0] | v[ca][1];
                    }
                    if (!any) continue;
                    bool range_ok = true;
                    for (int ca = 0; ca < CA; ++ca)
                        for (int r = 0; r < 2; ++r) range_ok = range_ok && v[ca][r] >= vmin && v[ca][r] <= vmax;
                    if (!range_ok) { bad.store(1); continue; }
                    for (int ca = 0; ca < CA; ++ca) my_nnz += (v[ca][0] != 0) + (v[ca][1] != 0);
                    const int kb = kk >> 5, t = (kk >> 3) & 3, j = kk & 7;
                    const int lane = 4 * g + t;
                    mask[(size_t)lane * nkb + kb] |= (uint8_t)(1u << j);
                    const size_t at = (size_t)lane * nkb * 8 + len[lane]++;
                    if (w2) {
                        stream[at] = (uint8_t)((v[0][0] + 2) | ((v[0][1] + 2) << 2) | ((v[1][0] + 2) << 4) | ((v[1][1] + 2) << 6));
                    } else {
                        stream[at] = (uint8_t)(((v[0][1] & 0xF) << 4) | ((v[0][0] + 8) & 0xF));
                        if (CA == 2) stream2[at] = (uint8_t)(((v[1][1] & 0xF) << 4) | ((v[1][0] + 8) & 0xF));
                    }
                }
            }
            int maxlen = 0;
            for (int l = 0; l < 32; ++l) { maxlen = std::max(maxlen, len[l]); my_P += len[l]; }
            const int J = (maxlen + 3) / 4;
            std::vector<uint8_t>& b = blobs[rb * h.n_segs + sg];
            // payload rows of 32 lane words; with C_A = 2 the rows of the two streams alternate
            b.assign((size_t)mask_bytes + (size_t)J * 128 * SR, 0);
            for (int l = 0; l < 32; ++l) {
                for (int w = 0; w < mask_rows; ++w)
                    std::memcpy(&b[(size_t)w * 128 + l * 4], &mask[(size_t)l * nkb + 4 * w], 4);
                const uint8_t* s = &stream[(size_t)l * nkb * 8];
                for (int i = 0; i < len[l]; ++i)
                    b[(size_t)mask_bytes + (size_t)(i >> 2) * 128 * SR + l * 4 + (i & 3)] = s[i];
                if (SR == 2) {
                    const uint8_t* s2 = &stream2[(size_t)l * nkb * 8];
                    for (int i = 0; i < len[l]; ++i)
                        b[(size_t)mask_bytes + (size_t)(i >> 2) * 256 + 128 + l * 4 + (i & 3)] = s2[i];
                }
            }
        }
        nnz += my_nnz;
        sum_P += my_P;
    });
    if (bad.load()) { h = HostMatrix(); return US_ERR_VALUE_RANGE; }

    // ---- offsets and the contiguous blob -------------------------------------------------
    h.item_off.assign(h.n_items + 1, 0);
    uint64_t off16 = 0;
    for (int64_t t = 0; t < h.n_items; ++t) {
        h.item_off[t] = (uint32_t)off16;
        off16 += blobs[t].size() / 16;
        h.max_item_bytes = std::max<uint32_t>(h.max_item_bytes, (uint32_t)blobs[t].size());
        if (off16 > 0xFFFFFFFFull) { h = HostMatrix(); return US_ERR_ALLOC; }
    }
    h.item_off[h.n_items] = (uint32_t)off16;
    try {
        h.blob.assign((size_t)off16 * 16, 0);
    } catch (...) {
        h = HostMatrix();
        return US_ERR_ALLOC;
    }
    parallel_for(h.n_items, threads, [&](int64_t t, int) {
        std::memcpy(h.blob.data() + (size_t)h.item_off[t] * 16, blobs[t].data(), blobs[t].size());
        std::vector<uint8_t>().swap(blobs[t]);
    });
    h.nnz = nnz.load();
    h.sum_P = sum_P.load();
    h.bytes_payload_padded = (int64_t)h.blob.size() - h.n_items * mask_bytes;
    return US_OK;
}

void decode_host(const HostMatrix& h, int8_t* W_out)
{
    std::memset(W_out, 0, (size_t)(h.M * h.K));
    if (!h.kernel_layout) { decode_generic(h, W_out); return; }
    const int CA = h.fmt.C_A, nkb = h.nkb / CA, mask_rows = h.mask_rows, K_L = h.fmt.K_L, K_B = K_L / CA;
    for (int64_t t = 0; t < h.n_items; ++t) {
        const int64_t rb = t / h.n_segs, sg = t % h.n_segs;
        const uint8_t* b = h.blob.data() + (size_t)h.item_off[t] * 16;
        const uint8_t* pay = b + (size_t)mask_rows * 128;
        for (int lane = 0; lane < 32; ++lane) {
            const int g = lane >> 2, tt = lane & 3;
            const int32_t ra = h.row_order[rb * 16 + g], rbw = h.row_order[rb * 16 + g + 8];
            int pos = 0;  // byte position in the lane's stream
            for (int kb = 0; kb < nkb; ++kb) {
                const uint8_t m = b[(size_t)(kb >> 2) * 128 + lane * 4 + (kb & 3)];
                for (int j = 0; j < 8; ++j) {
                    if (!((m >> j) & 1)) continue;
                    for (int ca = 0; ca < CA; ++ca) {
                        const int64_t k = sg * K_L + (int64_t)ca * K_B + 32 * kb + 8 * tt + j;
                        if (k >= h.K) continue;
                        int lo, hi;
                        if (h.w2) {
                            const uint8_t v = pay[(size_t)(pos >> 2) * 128 + lane * 4 + (pos & 3)];
                            lo = (int)((v >> (4 * ca)) & 3) - 2;
                            hi = (int)((v >> (4 * ca + 2)) & 3) - 2;
                        } else {
                            const uint8_t v = pay[(size_t)(pos >> 2) * 128 * CA + 128 * ca + lane * 4 + (pos & 3)];
                            lo = (int)(v & 0xF) - 8;
                            hi = (v >> 4) >= 8 ? (int)(v >> 4) - 16 : (int)(v >> 4);
                        }
                        if (ra >= 0) W_out[(int64_t)ra * h.K + k] = (int8_t)lo;
                        if (rbw >= 0) W_out[(int64_t)rbw * h.K + k] = (int8_t)hi;
                    }
                    ++pos;
                }
            }
        }
    }
}

void fill_stats(const HostMatrix& h, us_stats* st)
{
    const int Q = h.fmt.R_A * h.fmt.C_A;
    st->M = h.M; st->K = h.K; st->Mp = h.Mp; st->Kp = h.Kp;
    st->nnz = h.nnz;
    st->sum_P = h.sum_P;
    const int bits = h.w2 ? 2 : 4;
    st->bytes_payload = ((int64_t)Q * h.sum_P * bits + 7) / 8;
    st->weight_bits = bits;
    st->reserved = 0;
    if (h.kernel_layout) {
        st->n_tiles = h.n_items;
        st->bytes_payload_padded = h.bytes_payload_padded;
        st->bytes_bitmap = h.n_items * (int64_t)h.mask_rows * 128;
        st->bytes_offsets = 4 * (h.n_items + 1);
    } else {
        st->n_tiles = h.gen.n_lt;
        st->bytes_payload_padded = (int64_t)h.gen.values.size();
        st->bytes_bitmap = 8 * h.gen.n_lt * h.gen.words_per_lt;
        st->bytes_offsets = 4 * (h.gen.n_lt + 1);
    }
    st->bytes_total = st->bytes_payload_padded + st->bytes_bitmap + st->bytes_offsets;
    st->pmr = (bits / 8.0) * (double)h.nnz / (double)(st->bytes_bitmap + st->bytes_offsets);
    st->fill = (double)Q * (double)h.sum_P / ((double)h.M * (double)h.K);
    st->fmt = h.fmt;
}

void make_schedule(const HostMatrix& h, int n_cta, int G, std::vector<uint32_t>* begin,
                   int* max_local_strips)
{
    // Processing order: K range kr (G segments, the last one possibly shorter), then strip, then
    // segment within the range. Position u of that order maps to tile rb * n_segs + kr * G + sgl.
    begin->assign((size_t)n_cta + 1, 0);
    const int64_t n_kr = (h.n_segs + G - 1) / G;
    // Cost of a tile in the balance: its bytes (units of 16) plus a constant. The decode works per
    // k-block, whatever the payload: a tile of a sparse strip takes nearly as long as one of a dense
    // strip, so balancing bytes alone overloads the CTAs that get the sparse strips. Measured on a
    // row-varying 4096 x 11008 matrix with sorted rows: N = 8 11.5 -> 10.0 us, N = 32 25.5 -> 20.3 us
    // with cost = bytes + 2 x the average tile; uniform matrices are unaffected.
    const uint64_t avg16 = std::max<uint64_t>(1, h.item_off[h.n_items] / (uint64_t)std::max<int64_t>(1, h.n_items));
    auto tile_cost = [&](uint32_t units16) -> uint64_t {
        return units16 + 2 * avg16;
    };
    std::vector<uint64_t> prefix((size_t)h.n_items + 1, 0);
    std::vector<int32_t> strip_of((size_t)h.n_items), kr_of((size_t)h.n_items);
    int64_t u = 0;
    for (int64_t kr = 0; kr < n_kr; ++kr) {
        const int64_t g_kr = std::min<int64_t>(G, h.n_segs - kr * G);
        for (int64_t rb = 0; rb < h.n_strips; ++rb)
            for (int64_t sgl = 0; sgl < g_kr; ++sgl, ++u) {
                const int64_t t = rb * h.n_segs + kr * G + sgl;
                prefix[u + 1] = prefix[u] + tile_cost(h.item_off[t + 1] - h.item_off[t]);
                strip_of[u] = (int32_t)rb;
                kr_of[u] = (int32_t)kr;
            }
    }
    const uint64_t total = prefix[h.n_items];
    // With one K range the cuts fall on strip boundaries: every strip is then summed inside one CTA
    // and nothing goes through the global split-K workspace at all; that is worth far more than the
    // finer byte balance of cutting inside strips (measured at N = 8: 11008 x 4096 11.2 -> 9.0 us,
    // 13824 x 5120 13.4 -> 11.2 us, 28672 x 8192 26.6 -> 25.0 us). With several K ranges every strip
    // goes through the workspace anyway and aligned cuts make no measurable difference.
    const bool whole_strips = n_kr == 1;
    const int64_t g_last = h.n_segs - (n_kr - 1) * G;
    int64_t pos = 0;
    // Tilt (per mille): CTA 0 gets that much more than the average share, the last CTA that much less,
    // linearly in between. On the B200 the CTAs with the highest block indices end last, launch after
    // launch (they land on the SMs whose tile copies take longest); 3 % of tilt takes 2 % off the
    // 28672 x 8192 case (25.0 -> 24.5 us), 6 % and more start to hurt other shapes, a negative tilt
    // costs 2 %.
    constexpr int tilt = 30;
    for (int c = 0; c <= n_cta; ++c) {
        // (only where a CTA's share is many strips: on small shares the rounding to strips decides)
        const double x = (double)c / (double)n_cta, a = (whole_strips && h.n_strips >= (int64_t)8 * n_cta) ? tilt * 1e-3 : 0.0;
        const uint64_t target = (uint64_t)((double)total * (x + a * x * (1.0 - x)));
        while (pos < h.n_items && prefix[pos] < target) ++pos;
        if (whole_strips && pos < h.n_items) {
            // round to the nearest strip boundary of the position's K range (in bytes)
            const int64_t kr = kr_of[pos];
            const int64_t base = kr * h.n_strips * G, g = (kr == n_kr - 1) ? g_last : G;
            const int64_t down = base + (pos - base) / g * g, up = std::min<int64_t>(h.n_items, down + g);
            pos = (prefix[pos] - prefix[down] <= prefix[up] - prefix[pos]) ? down : up;
        }
        (*begin)[c] = (uint32_t)std::max<int64_t>(pos, c ? (int64_t)(*begin)[c - 1] : 0);
    }
    (*begin)[n_cta] = (uint32_t)h.n_items;
    // Several K ranges: no CTA should straddle a range boundary -- changing range costs a CTA a full
    // restaging of X behind a CTA-wide barrier (about 9 K cycles), and the whole launch waits for
    // those few CTAs. Give every range a whole number of CTAs in proportion to its bytes and split
    // each range evenly among its own.
    // (Not with one-segment ranges -- the direct mode: there a range is small, changing it is cheap,
    // and rounding CTAs to many ranges unbalances them: N = 64 on 28672 x 8192 87 -> 93 us.)
    if (n_kr > 1 && G > 1 && n_kr * 8 <= n_cta) {
        std::vector<int64_t> r_beg((size_t)n_kr + 1, 0);
        for (int64_t kr = 0; kr < n_kr; ++kr) r_beg[kr + 1] = std::min<int64_t>(h.n_items, (kr + 1) * h.n_strips * G);
        r_beg[n_kr] = h.n_items;
        std::vector<int> n_of((size_t)n_kr, 1);
        int used = (int)n_kr;
        std::vector<double> want((size_t)n_kr);
        for (int64_t kr = 0; kr < n_kr; ++kr)
            want[kr] = (double)(prefix[r_beg[kr + 1]] - prefix[r_beg[kr]]) / (double)std::max<uint64_t>(1, total) * n_cta;
        while (used < n_cta) {   // one more CTA to the range that is furthest below its fair number
            int64_t best = 0;
            for (int64_t kr = 1; kr < n_kr; ++kr)
                if (want[kr] - n_of[kr] > want[best] - n_of[best]) best = kr;
            ++n_of[best];
            ++used;
        }
        int c = 0;
        for (int64_t kr = 0; kr < n_kr; ++kr) {
            const uint64_t b0 = prefix[r_beg[kr]], b1 = prefix[r_beg[kr + 1]];
            int64_t q = r_beg[kr];
            for (int i = 0; i < n_of[kr]; ++i, ++c) {
                const uint64_t target = b0 + (b1 - b0) * (uint64_t)i / (uint64_t)n_of[kr];
                while (q < r_beg[kr + 1] && prefix[q] < target) ++q;
                (*begin)[c] = (uint32_t)q;
            }
        }
        (*begin)[n_cta] = (uint32_t)h.n_items;
    }
    int worst = 1;
    for (int c = 0; c < n_cta; ++c) {
        int64_t a = (*begin)[c], b = (*begin)[c + 1];
        while (a < b) {  // one K range at a time
            int64_t e = a;
            while (e < b && kr_of[e] == kr_of[a]) ++e;
            worst = std::max(worst, strip_of[e - 1] - strip_of[a] + 1);
            a = e;
        }
    }
    if (max_local_strips) *max_local_strips = worst;
}

}  // namespace us
