// Set-up kernels: the count table N(n,k) (Sec. 2.4, App. C.2 / Algorithm 4) and
// the amplitude codebook (Sec. 3.4).  Both are cold: they run once per (N,K)
// or per (N,G,b).
#include "mp_uint.cuh"
#include "pvq_internal.cuh"
#include "pvq_search.cuh"

namespace pvq {

// ------------------------------------------------------------- count table
//
// One thread block, thread k owns column k and keeps N(n,k) in registers while
// the block walks the rows n = 0, 1, ...:
//   a_k = N(n-1,k) + N(n-1,k-1)   (the diagonal term, from the neighbour's value)
//   N(n,k) = sum_{i<=k} a_i, a_0 = 1   (inclusive prefix sum over k)
// which is the recurrence N(n,k) = N(n-1,k) + N(n,k-1) + N(n-1,k-1) unrolled
// along k.  The prefix sum is a Hillis-Steele scan through shared memory.  A
// table of this size never needs more than one block, so there is no
// inter-block barrier.
// W is the width the kernel computes in, Wc <= W the words of an entry in memory.
template <int W>
__global__ void __launch_bounds__(1024) count_table_kernel(int N, int K, int Wc, uint32_t* __restrict__ table) {
    extern __shared__ uint32_t sm[];  // two buffers of (K+1) entries of W words
    const int k = threadIdx.x;
    const int KP = K + 1;
    uint32_t* buf0 = sm;
    uint32_t* buf1 = sm + static_cast<size_t>(KP) * W;
    const bool live = k < KP;

    mp<W> v;  // N(n,k) for the current row
    mp_zero(v);
    if (k == 0) v.w[0] = 1u;  // row 0: N(0,0) = 1, N(0,k>=1) = 0

    for (int n = 0; n < N; ++n) {
        if (live) {
#pragma unroll
            for (int w = 0; w < W; ++w)
                if (w < Wc) table[(static_cast<size_t>(n) * KP + k) * Wc + w] = v.w[w];
#pragma unroll
            for (int w = 0; w < W; ++w) buf0[k * W + w] = v.w[w];
        }
        __syncthreads();
        // a_k = N(n,k) + N(n,k-1) for the next row; a_0 = 1
        if (live) {
            if (k == 0) {
                mp_zero(v);
                v.w[0] = 1u;
            } else {
                mp<W> left = mp_load<W>(buf0 + (k - 1) * W);
                mp_add<W>(v, left);
            }
        }
        __syncthreads();
        // inclusive scan of a over k
        uint32_t* src = buf0;
        uint32_t* dst = buf1;
        for (int off = 1; off < KP; off <<= 1) {
            if (live) {
#pragma unroll
                for (int w = 0; w < W; ++w) src[k * W + w] = v.w[w];
            }
            __syncthreads();
            if (live && k >= off) {
                mp<W> o = mp_load<W>(src + (k - off) * W);
                mp_add<W>(v, o);
            }
            uint32_t* t = src;
            src = dst;
            dst = t;
        }
        __syncthreads();
    }
}

// The same table for more pulses than a block has threads (K up to kMaxPulses), built by many
// blocks (App. C.2 / Algorithm 4 spreads a row over blocks and puts a barrier between rows).
// Row n is the inclusive prefix sum over k of a_k = N(n-1,k) + N(n-1,k-1), read back from the
// row before it.  Thread t of the launch owns the `chunk` consecutive columns from t * chunk.
// Two launches per row, the launch boundary being the barrier between blocks (every wait is
// the stream's: nothing spins):
//   count_row_sums_kernel   every block sums the a_k of its columns and writes the total;
//   count_row_write_kernel  every block scans the totals of the blocks before it, scans its
//                           threads' sums once more, and writes its columns of the row.
// The block totals go to a scratch area inside the blob that a later set-up kernel overwrites.

// Inclusive scan over the block's threads of one W-word value each, through `buf`
// (blockDim.x entries of W words); on return buf[t] holds thread t's result as well.
template <int W>
__device__ __forceinline__ void block_scan_inclusive(mp<W>& v, uint32_t* buf) {
    const int t = threadIdx.x;
#pragma unroll
    for (int w = 0; w < W; ++w) buf[t * W + w] = v.w[w];
    __syncthreads();
    for (int off = 1; off < static_cast<int>(blockDim.x); off <<= 1) {
        mp<W> o;
        mp_zero(o);
        if (t >= off) o = mp_load<W>(buf + (t - off) * W);
        __syncthreads();
        mp_add<W>(v, o);
#pragma unroll
        for (int w = 0; w < W; ++w) buf[t * W + w] = v.w[w];
        __syncthreads();
    }
}

// sum of a_k over the columns [k0, k1) of a thread
template <int W>
__device__ __forceinline__ mp<W> chunk_sum(const uint32_t* __restrict__ prev, int Wc, int k0, int k1) {
    mp<W> run;
    mp_zero(run);
    for (int k = k0; k < k1; ++k) {
        for (int j = (k > 0 ? k - 1 : k); j <= k; ++j) {
            mp<W> v;
#pragma unroll
            for (int w = 0; w < W; ++w) v.w[w] = w < Wc ? prev[static_cast<size_t>(j) * Wc + w] : 0u;
            mp_add<W>(run, v);
        }
    }
    return run;
}

__global__ void count_row0_kernel(int K, int Wc, uint32_t* __restrict__ table) {
    const size_t words = static_cast<size_t>(K + 1) * Wc;  // row 0: N(0,0) = 1, N(0,k>=1) = 0
    for (size_t i = blockIdx.x * blockDim.x + threadIdx.x; i < words; i += static_cast<size_t>(gridDim.x) * blockDim.x)
        table[i] = i == 0 ? 1u : 0u;
}

template <int W>
__global__ void __launch_bounds__(256) count_row_sums_kernel(const uint32_t* __restrict__ prev, int KP, int Wc, int chunk,
                                                             uint32_t* __restrict__ block_totals) {
    extern __shared__ uint32_t buf[];  // blockDim.x entries of W words
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int k0 = min(t * chunk, KP), k1 = min(k0 + chunk, KP);
    mp<W> v = chunk_sum<W>(prev, Wc, k0, k1);
    block_scan_inclusive<W>(v, buf);
    if (threadIdx.x == blockDim.x - 1) {
#pragma unroll
        for (int w = 0; w < W; ++w) block_totals[blockIdx.x * W + w] = v.w[w];
    }
}

template <int W>
__global__ void __launch_bounds__(256) count_row_write_kernel(const uint32_t* __restrict__ prev, uint32_t* __restrict__ cur,
                                                              int KP, int Wc, int chunk,
                                                              const uint32_t* __restrict__ block_totals) {
    extern __shared__ uint32_t buf[];
    // everything in the blocks before this one (gridDim.x <= blockDim.x: one total per thread)
    mp<W> base;
    mp_zero(base);
    if (threadIdx.x < gridDim.x) base = mp_load<W>(block_totals + threadIdx.x * W);
    block_scan_inclusive<W>(base, buf);
    mp_zero(base);
    if (blockIdx.x > 0) base = mp_load<W>(buf + (blockIdx.x - 1) * W);
    __syncthreads();  // buf is reused below
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int k0 = min(t * chunk, KP), k1 = min(k0 + chunk, KP);
    mp<W> v = chunk_sum<W>(prev, Wc, k0, k1);
    block_scan_inclusive<W>(v, buf);
    if (threadIdx.x > 0) mp_add<W>(base, mp_load<W>(buf + (threadIdx.x - 1) * W));  // the threads before this one
    for (int k = k0; k < k1; ++k) {
        mp_add<W>(base, chunk_sum<W>(prev, Wc, k, k + 1));
        for (int w = 0; w < Wc; ++w) cur[static_cast<size_t>(k) * Wc + w] = base.w[w];
    }
}

// The other sections of the blob (TableLayout): the same numbers re-laid for the decode walk,
// narrow copies saturated at their width, and N(N,K) itself.
// with_enc == 0: the encoder's cumulative tables are written by derive_enc_tables_kernel instead.
template <int W>
__global__ void derive_tables_kernel(int N, int K, int Wc, uint32_t* __restrict__ blob, int with_enc) {
    const TableLayout L = table_layout(N, K, Wc);
    if (L.rowlen == 0) return;
    const int KP = K + 1;
    const int entries = N * L.rowlen;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < entries; e += gridDim.x * blockDim.x) {
        const int i = e / L.rowlen;
        const int col = e - i * L.rowlen;
        const bool pad = col > K;  // never read; filled with all ones
        uint32_t v[W];
#pragma unroll
        for (int w = 0; w < W; ++w)
            v[w] = pad ? 0xffffffffu : (w < Wc ? blob[(static_cast<size_t>(N - 1 - i) * KP + col) * Wc + w] : 0u);
        uint32_t* top = blob + L.walk_off[0] / 4 + static_cast<size_t>(e) * L.top_words;
        for (int w = 0; w < L.top_words; ++w) top[w] = w < W ? v[w] : 0u;
        if (L.walk_bytes[1]) {  // two-word copy: values from 2^62 up become 2^62
            uint32_t hi = 0;
#pragma unroll
            for (int w = 2; w < W; ++w) hi |= v[w];
            const uint32_t v1 = W > 1 ? v[W > 1 ? 1 : 0] : 0u;
            const bool big = pad || hi != 0u || (v1 >> 30) != 0u;
            uint32_t* t2 = blob + L.walk_off[1] / 4 + static_cast<size_t>(e) * 2;
            t2[0] = big ? 0u : v[0];
            t2[1] = big ? 0x40000000u : v1;
        }
        if (L.walk_bytes[2]) {  // one-word copy: values from 2^30 up become 2^30
            uint32_t hi = 0;
#pragma unroll
            for (int w = 1; w < W; ++w) hi |= v[w];
            const bool big = pad || hi != 0u || (v[0] >> 30) != 0u;
            blob[L.walk_off[2] / 4 + e] = big ? 0x40000000u : v[0];
        }
    }
    // encoder tables: one thread per position runs the prefix sum V(n,k) = V(n,k-1) + N(n,k)
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; with_enc && i < N; i += gridDim.x * blockDim.x) {
        const uint32_t* row = blob + static_cast<size_t>(N - 1 - i) * KP * Wc;
        const int TW = L.top_words;
        uint32_t* eu = blob + L.enc_off[0] / 4 + static_cast<size_t>(i) * (K + 2) * TW;
        uint32_t* e2 = blob + L.enc_off[1] / 4 + static_cast<size_t>(i) * (K + 2) * TW;
        uint32_t* ev = blob + L.enc_off[2] / 4 + static_cast<size_t>(i) * (K + 2) * TW;
        uint32_t v[W], vprev[W];
#pragma unroll
        for (int w = 0; w < W; ++w) v[w] = vprev[w] = 0u;
        for (int c = -1; c <= K; ++c) {
            if (c >= 0) {
#pragma unroll
                for (int w = 0; w < W; ++w) vprev[w] = v[w];
                unsigned long long carry = 0;
#pragma unroll
                for (int w = 0; w < W; ++w) {
                    const uint32_t add = w < Wc ? row[c * Wc + w] : 0u;
                    const unsigned long long sum = static_cast<unsigned long long>(v[w]) + add + carry;
                    v[w] = w < Wc ? static_cast<uint32_t>(sum) : 0u;  // modulo 2^(32 Wc)
                    carry = sum >> 32;
                }
            }
            unsigned long long cu = 0, c2 = 0;
            for (int w = 0; w < TW; ++w) {
                const uint32_t a = w < W ? v[w < W ? w : 0] : 0u, bprev = w < W ? vprev[w < W ? w : 0] : 0u;
                const unsigned long long su = static_cast<unsigned long long>(a) + bprev + cu;
                const unsigned long long s2 = static_cast<unsigned long long>(a) + a + c2;
                cu = su >> 32;
                c2 = s2 >> 32;
                const bool in = w < Wc;  // words beyond Wc stay zero: the sums are kept modulo 2^(32 Wc)
                eu[(c + 1) * TW + w] = in ? static_cast<uint32_t>(su) : 0u;
                e2[(c + 1) * TW + w] = in ? static_cast<uint32_t>(s2) : 0u;
                ev[(c + 1) * TW + w] = a;
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // N(N,K) = N(N-1,K) + 2 sum_{j=1..K} N(N-1,K-j)   (every point of P(N,K) by its first
        // coordinate: 0, or +-j with K-j pulses left for the other N-1)
        constexpr int BW = bound_words_of(W);
        uint32_t acc[BW];
        for (int w = 0; w < BW; ++w) acc[w] = 0u;
        const uint32_t* row = blob + static_cast<size_t>(N - 1) * KP * Wc;
        for (int col = 0; col <= K; ++col) {
            const int times = col == K ? 1 : 2;
            for (int rep = 0; rep < times; ++rep) {
                unsigned long long carry = 0;
                for (int w = 0; w < BW; ++w) {
                    const unsigned long long add = w < Wc ? row[col * Wc + w] : 0u;
                    const unsigned long long sum = static_cast<unsigned long long>(acc[w]) + add + carry;
                    acc[w] = static_cast<uint32_t>(sum);
                    carry = sum >> 32;
                }
            }
        }
        for (int w = 0; w < BW; ++w) blob[L.bound_off / 4 + w] = acc[w];
    }
}

// The sections for the shared-memory kernels (see TableLayout): the walk table as doubles,
// and the encoder's telescoped tables with the value the sum starts from.  Runs after
// derive_tables_kernel: it reads the walk table and the cumulative tables U and 2V.
__global__ void derive_fast_tables_kernel(int N, int K, int Wc, uint32_t* __restrict__ blob) {
    const TableLayout L = table_layout(N, K, Wc);
    if (L.walkd_bytes == 0) return;
    const int TW = L.top_words;
    const int entries = N * L.rowlen;
    const int tid = blockIdx.x * blockDim.x + threadIdx.x, nthr = gridDim.x * blockDim.x;
    double* wd = reinterpret_cast<double*>(blob + L.walkd_off / 4);
    for (int e = tid; e < entries; e += nthr) {
        const uint32_t* t = blob + L.walk_off[0] / 4 + static_cast<size_t>(e) * TW;
        uint32_t hi = 0;
        for (int w = 2; w < TW; ++w) hi |= t[w];
        const uint32_t t1 = TW > 1 ? t[1] : 0u;
        const bool big = hi != 0u || (t1 >> 21) != 0u;  // 2^53 and up (the row padding too)
        const unsigned long long v = static_cast<unsigned long long>(t[0]) | (static_cast<unsigned long long>(t1) << 32);
        wd[e] = big ? 9007199254740992.0 : static_cast<double>(v);  // exact: below 2^53
    }
    const uint32_t* U = blob + L.enc_off[0] / 4;  // (i, col + 1), K + 2 entries a row
    const uint32_t* V2 = blob + L.enc_off[1] / 4;
    if (tid < TW) blob[L.start_off / 4 + tid] = U[static_cast<size_t>(K + 1) * TW + tid];  // U(N-1, K): position 0
    if (L.cenc_bytes == 0) return;
    const int centries = N * L.crow;
    for (int e = tid; e < centries; e += nthr) {
        const int i = e / L.crow;
        const int k = e - i * L.crow;
        // a row is TW planes of crow words: word w of entry k at (i * TW + w) * crow + k
        uint32_t* c0 = blob + L.cenc_off[0] / 4 + static_cast<size_t>(i) * TW * L.crow + k;
        uint32_t* c1 = blob + L.cenc_off[1] / 4 + static_cast<size_t>(i) * TW * L.crow + k;
        if (k > K) {  // the rest of the row
            for (int w = 0; w < TW; ++w) c0[w * L.crow] = c1[w * L.crow] = 0u;
            continue;
        }
        const uint32_t* un = U + (static_cast<size_t>(i + 1) * (K + 2) + k + 1) * TW;  // U(n-1, k): next position
        const uint32_t* u = U + (static_cast<size_t>(i) * (K + 2) + k + 1) * TW;
        const uint32_t* v2 = V2 + (static_cast<size_t>(i) * (K + 2) + k + 1) * TW;
        long long b0 = 0, b1 = 0;  // borrows
        for (int w = 0; w < TW; ++w) {
            const long long a = (i + 1 < N && w < Wc) ? static_cast<long long>(un[w]) : 0;
            const long long d0 = a - static_cast<long long>(u[w]) + b0;
            const long long d1 = a - static_cast<long long>(v2[w]) + b1;
            b0 = d0 >> 32;  // 0 or -1
            b1 = d1 >> 32;
            const bool in = w < Wc;  // modulo 2^(32 Wc): the words above stay zero
            c0[w * L.crow] = in ? static_cast<uint32_t>(d0) : 0u;
            c1[w * L.crow] = in ? static_cast<uint32_t>(d1) : 0u;
        }
    }
}

// The search section (SearchLayout), block n = row n, thread m = threshold m.  Runs after
// derive_tables_kernel: thresholds and increments come from the cumulative tables U and 2V.
// The bucket table of a row holds, for every bucket, how many thresholds lie in earlier
// buckets, and the low key bits of the threshold in the bucket, if any: thread m writes the
// buckets after that of threshold m-1 up to its own.
__global__ void __launch_bounds__(256) derive_search_tables_kernel(int N, int K, int Wc, uint32_t* __restrict__ blob,
                                                                   const __grid_constant__ SearchLayout S) {
    __shared__ uint32_t bucket_of[256];
    const TableLayout L = table_layout(N, K, Wc);
    const int TW = L.top_words;  // words per entry of the cumulative tables
    const int n = blockIdx.x, m = threadIdx.x;
    const int i = N - 1 - n;     // the position whose row of the cumulative tables this is
    const int k = m >> 1;
    const int last = n == 0 ? 1 : 2 * K;  // thresholds of the row: 0..last
    const int RW = S.rows.words[n];       // words of this row's arithmetic: its planes
    uint8_t* sec = reinterpret_cast<uint8_t*>(blob) + S.off;
    const uint32_t* U = blob + L.enc_off[0] / 4;   // (i, col + 1), K + 2 entries a row
    const uint32_t* V2 = blob + L.enc_off[1] / 4;
    uint32_t t[4] = {0u, 0u, 0u, 0u};
    if (m <= 2 * K) {
        const uint32_t* src = ((m & 1) ? V2 : U) + (static_cast<size_t>(i) * (K + 2) + k + 1) * TW;
        for (int w = 0; w < Wc; ++w) t[w] = src[w];
    }
    if (m < 2 * K + 2) {
        const size_t at = S.rows.te_off[n] / 4u + static_cast<size_t>(m);  // word 0; word w is w planes further
        uint32_t* T = reinterpret_cast<uint32_t*>(sec + S.t_off) + at;
        uint32_t* E = reinterpret_cast<uint32_t*>(sec + S.e_off) + at;
        // E = U(n-1, k) - T, modulo 2^(32 RW); U(-1, .) = 0
        const uint32_t* un = U + (static_cast<size_t>(i + 1) * (K + 2) + k + 1) * TW;
        long long borrow = 0;
        for (int w = 0; w < RW; ++w) {
            const long long a = (n >= 1 && w < Wc && m <= 2 * K) ? static_cast<long long>(un[w]) : 0;
            const long long d = a - static_cast<long long>(w < Wc ? t[w] : 0u) + borrow;
            borrow = d >> 32;  // 0 or -1
            T[static_cast<size_t>(w) * S.plane] = t[w];
            E[static_cast<size_t>(w) * S.plane] = static_cast<uint32_t>(d);
        }
    }
    const uint32_t sh = S.rows.shift[n];  // 1..23
    const uint32_t key = search_key(t, Wc);
    bucket_of[m] = m <= last ? (key >> sh) - (kSearchKeyOfOne >> sh) : 0u;
    __syncthreads();
    if (m <= last) {
        uint32_t* B = reinterpret_cast<uint32_t*>(sec + S.b_off) + S.rows.b_off[n];
        const uint32_t hi = bucket_of[m];
        const uint32_t lo = m == 0 ? 0u : bucket_of[m - 1] + 1u;
        // a threshold below 2^24 is its key: equal key bits then mean equal numbers, and bit 8
        // of the entry says so (it keeps the decoder from comparing in full)
        const uint32_t exact = key < 0x4b800000u ? 0x100u : 0u;
        for (uint32_t b = lo; b <= hi && b < S.rows.b_len[n]; ++b)
            B[b] = (b == hi ? (key << (32u - sh)) | exact : 0xffffff00u) | static_cast<uint32_t>(m);
    }
    if (m == 0) {
        uint32_t* rec = reinterpret_cast<uint32_t*>(sec + S.rec_off) + 4 * n;
        rec[0] = 32u - sh;
        rec[1] = S.e_off + S.rows.te_off[n];
        rec[2] = S.b_off + 4u * (S.rows.b_off[n] - (kSearchKeyOfOne >> sh));
        rec[3] = sh;
        if (n == 0) {
            uint32_t* head = reinterpret_cast<uint32_t*>(sec);
            head[0] = kSearchMagic;
            head[1] = static_cast<uint32_t>(N);
            head[2] = static_cast<uint32_t>(K);
            head[3] = S.total;
            for (int w = 4; w >= 1; --w) head[8 - w] = static_cast<uint32_t>(S.count[w]);
        }
    }
}

static int launch_search_tables(int N, int K, int Wc, uint32_t* d_table, cudaStream_t s) {
    const SearchLayout& S = search_layout_for(N, K);
    if (!S.present) return PVQ_OK;
    derive_search_tables_kernel<<<N, 256, 0, s>>>(N, K, Wc, d_table, S);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

template <int W>
static int launch_count_table(int N, int K, int Wc, uint32_t* d_table, cudaStream_t s) {
    const int threads = ((K + 1 + 31) / 32) * 32;
    const size_t smem = 2u * static_cast<size_t>(K + 1) * W * sizeof(uint32_t);
    DeviceInfo di;
    const int st = device_info(&di);
    if (st != PVQ_OK) return st;
    if (smem > static_cast<size_t>(di.smem_max)) return PVQ_ERR_UNSUPPORTED;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(count_table_kernel<W>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return set_cuda_error(e);
    }
    count_table_kernel<W><<<1, threads, smem, s>>>(N, K, Wc, d_table);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_cuda_error(e);
    if (table_layout(N, K, Wc).rowlen != 0) {
        derive_tables_kernel<W><<<16, 256, 0, s>>>(N, K, Wc, d_table, 1);
        if ((e = cudaGetLastError()) != cudaSuccess) return set_cuda_error(e);
        derive_fast_tables_kernel<<<16, 256, 0, s>>>(N, K, Wc, d_table);
        if ((e = cudaGetLastError()) != cudaSuccess) return set_cuda_error(e);
        return launch_search_tables(N, K, Wc, d_table, s);
    }
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

// The encoder's cumulative tables entry by entry, for tables too large for the one-thread-per-row
// prefix sums of derive_tables_kernel.  With V(n,k) = sum_{j<=k} N(n,j):
//   U(n,k) = V(n,k) + V(n,k-1) = N(n+1,k)     (the recurrence of Sec. 2.4 summed over k)
//   N(n,k) = V(n,k) - V(n,k-1),  so  2 V(n,k) = N(n+1,k) + N(n,k)
// Row n + 1 is the next row of the count table, for n = N-1 the row `row_n` that the builder
// ran one row further (N(N,k), modulo 2^(32 Wc): top_overflow says that N(N,K) is exactly
// 2^(32 Wc), the one value that does not fit).
template <int W>
__global__ void derive_enc_tables_kernel(int N, int K, int Wc, uint32_t* __restrict__ blob,
                                         const uint32_t* __restrict__ row_n, int top_overflow) {
    const TableLayout L = table_layout(N, K, Wc);
    const int TW = L.top_words;
    const int KP = K + 1;
    const long long entries = static_cast<long long>(N) * (K + 2);
    for (long long e = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; e < entries;
         e += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int i = static_cast<int>(e / (K + 2));
        const int c = static_cast<int>(e - static_cast<long long>(i) * (K + 2)) - 1;  // -1..K
        const int n = N - 1 - i;
        uint32_t* eu = blob + L.enc_off[0] / 4 + static_cast<size_t>(e) * TW;
        uint32_t* e2 = blob + L.enc_off[1] / 4 + static_cast<size_t>(e) * TW;
        uint32_t* ev = blob + L.enc_off[2] / 4 + static_cast<size_t>(e) * TW;
        const uint32_t* up = c < 0 ? nullptr : (n + 1 < N ? blob + (static_cast<size_t>(n + 1) * KP + c) * Wc
                                                         : row_n + static_cast<size_t>(c) * Wc);
        const uint32_t* np = c < 0 ? nullptr : blob + (static_cast<size_t>(n) * KP + c) * Wc;
        unsigned long long carry = 0;
        uint32_t sum[W + 1];  // U + N = 2 V, one word more than an entry
#pragma unroll
        for (int w = 0; w < W; ++w) {
            const unsigned long long a = (up && w < Wc) ? up[w] : 0u, b = (np && w < Wc) ? np[w] : 0u;
            const unsigned long long t = a + b + carry;
            sum[w] = static_cast<uint32_t>(t);
            carry = t >> 32;
        }
        sum[W] = static_cast<uint32_t>(carry);
        // the word above the entry: a carry out of Wc words sits in sum[Wc]; the lost top bit of U adds one
        uint32_t above = Wc < W ? sum[Wc] : sum[W];
        if (top_overflow && i == 0 && c == K) above += 1u;
        for (int w = 0; w < TW; ++w) {
            const bool in = w < Wc;
            const uint32_t hi = w + 1 < Wc ? sum[w + 1 < W ? w + 1 : W] : above;  // the word above word w of 2 V
            eu[w] = (in && up) ? up[w] : 0u;
            e2[w] = in ? sum[w < W ? w : W] : 0u;
            ev[w] = in ? (sum[w < W ? w : W] >> 1) | (hi << 31) : 0u;
        }
    }
}

template <int W>
static int launch_count_table_chunked(int N, int K, int Wc, uint32_t* d_table, cudaStream_t s) {
    const TableLayout L = table_layout(N, K, Wc);
    DeviceInfo di;
    int st = device_info(&di);
    if (st != PVQ_OK) return st;
    const int threads = 256;
    const int KP = K + 1;
    const int chunk = (KP + di.sms * threads - 1) / (di.sms * threads);  // at most one block per SM
    const int blocks = (KP + chunk * threads - 1) / (chunk * threads);   // <= threads, as the write kernel needs
    const size_t smem = static_cast<size_t>(threads) * W * sizeof(uint32_t);
    constexpr size_t kScratchRowOffset = 32768;  // behind the totals (at most 256 blocks of 32 words)
    // the block totals: at the start of the decoder's first table, which derive_tables_kernel fills below
    if (L.rowlen == 0 || static_cast<size_t>(blocks) * W * 4u > L.walk_bytes[0] || blocks > threads)
        return PVQ_ERR_UNSUPPORTED;
    uint32_t* totals = d_table + L.walk_off[0] / 4;
    count_row0_kernel<<<16, 256, 0, s>>>(K, Wc, d_table);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_cuda_error(e);
    for (int n = 1; n < N; ++n) {
        const uint32_t* prev = d_table + static_cast<size_t>(n - 1) * KP * Wc;
        uint32_t* cur = d_table + static_cast<size_t>(n) * KP * Wc;
        count_row_sums_kernel<W><<<blocks, threads, smem, s>>>(prev, KP, Wc, chunk, totals);
        count_row_write_kernel<W><<<blocks, threads, smem, s>>>(prev, cur, KP, Wc, chunk, totals);
        if ((e = cudaGetLastError()) != cudaSuccess) return set_cuda_error(e);
    }
    // One row more, N(N,k), behind the totals in the same scratch area: with it the encoder's
    // cumulative tables follow entry by entry.  (Where the area is too small the set-up kernel
    // below runs its own prefix sums.)
    const size_t row_bytes = static_cast<size_t>(KP) * Wc * 4u;
    const bool enc_by_entry = kScratchRowOffset + row_bytes <= L.walk_bytes[0];
    if (enc_by_entry) {
        const uint32_t* prev = d_table + static_cast<size_t>(N - 1) * KP * Wc;
        uint32_t* row_n = totals + kScratchRowOffset / 4;
        count_row_sums_kernel<W><<<blocks, threads, smem, s>>>(prev, KP, Wc, chunk, totals);
        count_row_write_kernel<W><<<blocks, threads, smem, s>>>(prev, row_n, KP, Wc, chunk, totals);
        derive_enc_tables_kernel<W><<<4 * di.sms, 256, 0, s>>>(N, K, Wc, d_table, row_n, count_fills_its_words(N, K) ? 1 : 0);
        if ((e = cudaGetLastError()) != cudaSuccess) return set_cuda_error(e);
    }
    derive_tables_kernel<W><<<4 * di.sms, 256, 0, s>>>(N, K, Wc, d_table, enc_by_entry ? 0 : 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return set_cuda_error(e);
    derive_fast_tables_kernel<<<16, 256, 0, s>>>(N, K, Wc, d_table);
    e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}

// ---------------------------------------------------------- scale codebook
//
// u = ||x_g||^2 / ||x_row||^2 ~ Beta(a, b) with a = N/2, b = N(G-1)/2, both
// integers for even N.  For integer parameters the CDF is a binomial tail:
//   I_x(a,b) = P[ Bin(n, x) >= a ],  n = a + b - 1
//            = 1 - sum_{j<a} C(n,j) x^j (1-x)^(n-j),
// a sum of a <= N/2 positive terms, evaluated in fp64.  The quantile is found
// by bisection on x until the bracket is one fp64 spacing wide.
__device__ double beta_cdf_int(double x, int a, int n) {
    if (x <= 0.0) return 0.0;
    if (x >= 1.0) return 1.0;
    double t = exp(static_cast<double>(n) * log1p(-x));  // (1-x)^n
    const double ratio = x / (1.0 - x);
    double sum = 0.0;
    for (int j = 0; j < a; ++j) {
        sum += t;
        t = t * (static_cast<double>(n - j) / static_cast<double>(j + 1)) * ratio;
    }
    return 1.0 - sum;
}

__device__ double beta_ppf_int(double p, int a, int n) {
    double lo = 0.0, hi = 1.0;
    for (int it = 0; it < 1100; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (mid <= lo || mid >= hi) break;
        if (beta_cdf_int(mid, a, n) < p)
            lo = mid;
        else
            hi = mid;
    }
    return 0.5 * (lo + hi);
}

__global__ void scale_codebook_kernel(int a, int n, int scale_bits, float* __restrict__ edges,
                                      float* __restrict__ levels) {
    const int L = 1 << scale_bits;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < L - 1) {
        if (edges) edges[t] = static_cast<float>(beta_ppf_int(static_cast<double>(t + 1) / L, a, n));
    } else if (t < 2 * L - 1) {
        const int q = t - (L - 1);
        if (levels) levels[q] = static_cast<float>(sqrt(beta_ppf_int((q + 0.5) / L, a, n)));
    }
}

}  // namespace pvq

using namespace pvq;

extern "C" int pvq_build_count_table(int N, int K, uint32_t* d_table, size_t bytes, pvq_stream_t stream) {
    if (!d_table || N < 1 || K < 1) return PVQ_ERR_INVALID_ARG;
    if (N > 256 || K > kMaxPulses) return PVQ_ERR_UNSUPPORTED;
    const int W = code_words_for(N, K);
    if (W == 0) return PVQ_ERR_INVALID_ARG;
    if (W > kMaxWords) return PVQ_ERR_UNSUPPORTED;
    if (!is_aligned(d_table, 16)) return PVQ_ERR_ALIGNMENT;
    if (bytes < pvq_count_table_bytes(N, K)) return PVQ_ERR_TABLE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // more pulses than threads of a block, or rows of 32 KB and more: the multi-block builder, in 8, 16 or 32 words
    if (K > 1023 || static_cast<long long>(K + 1) * W >= 8192) {
        if (W <= 8) return launch_count_table_chunked<8>(N, K, W, d_table, s);
        if (W <= 16) return launch_count_table_chunked<16>(N, K, W, d_table, s);
        return launch_count_table_chunked<32>(N, K, W, d_table, s);
    }
    switch (W) {
        case 1: return launch_count_table<1>(N, K, W, d_table, s);
        case 2: return launch_count_table<2>(N, K, W, d_table, s);
        case 3: return launch_count_table<3>(N, K, W, d_table, s);
        case 4: return launch_count_table<4>(N, K, W, d_table, s);
        case 5: return launch_count_table<5>(N, K, W, d_table, s);
        case 6: return launch_count_table<6>(N, K, W, d_table, s);
        case 7: return launch_count_table<7>(N, K, W, d_table, s);
        case 8: return launch_count_table<8>(N, K, W, d_table, s);
        case 9: return launch_count_table<9>(N, K, W, d_table, s);
        case 10: return launch_count_table<10>(N, K, W, d_table, s);
        case 11: return launch_count_table<11>(N, K, W, d_table, s);
        case 12: return launch_count_table<12>(N, K, W, d_table, s);
        default: break;
    }
    // wider codes: computed in the next of 16, 24, 32 words
    if (W <= 16) return launch_count_table<16>(N, K, W, d_table, s);
    if (W <= 24) return launch_count_table<24>(N, K, W, d_table, s);
    return launch_count_table<32>(N, K, W, d_table, s);
}

extern "C" int pvq_build_scale_codebook(int N, int64_t G, int scale_bits, float* d_edges, float* d_levels,
                                        pvq_stream_t stream) {
    if (N < 2 || (N & 1) || G < 2 || scale_bits < 1 || scale_bits > 8) return PVQ_ERR_INVALID_ARG;
    if (!d_edges && !d_levels) return PVQ_ERR_INVALID_ARG;
    const int64_t n64 = static_cast<int64_t>(N) * G / 2 - 1;  // a + b - 1
    if (n64 > (int64_t(1) << 30)) return PVQ_ERR_UNSUPPORTED;
    const int L = 1 << scale_bits;
    const int threads = 64;
    const int blocks = (2 * L - 1 + threads - 1) / threads;
    scale_codebook_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        N / 2, static_cast<int>(n64), scale_bits, d_edges, d_levels);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? PVQ_OK : set_cuda_error(e);
}
