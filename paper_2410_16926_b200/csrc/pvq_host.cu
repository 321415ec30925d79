// Host side of the C ABI: argument checks, exact integer helpers for choosing
// K (Sec. 3.3 Step 2), and translation of the public calls into kernel launches.
#include <algorithm>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>
#include <vector>

#include "pvq_internal.cuh"

namespace pvq {

static thread_local int g_last_cuda_error = 0;

int set_cuda_error(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return PVQ_ERR_CUDA;
}

bool is_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// ------------------------------------------------------------------ big ints
// Unsigned integers of up to kLimbs 32-bit limbs; only what choosing K needs.
namespace {

constexpr int kLimbs = 48;

struct BigU {
    uint32_t w[kLimbs];
    BigU() { std::memset(w, 0, sizeof w); }
    explicit BigU(uint32_t v) {
        std::memset(w, 0, sizeof w);
        w[0] = v;
    }
    // *this += o; false when the sum overflows kLimbs
    bool add(const BigU& o) {
        uint64_t c = 0;
        for (int i = 0; i < kLimbs; ++i) {
            uint64_t s = static_cast<uint64_t>(w[i]) + o.w[i] + c;
            w[i] = static_cast<uint32_t>(s);
            c = s >> 32;
        }
        return c == 0;
    }
    int bit_length() const {
        for (int i = kLimbs - 1; i >= 0; --i)
            if (w[i]) return 32 * i + (32 - __builtin_clz(w[i]));
        return 0;
    }
    bool is_pow2() const {
        int ones = 0;
        for (int i = 0; i < kLimbs; ++i) ones += __builtin_popcount(w[i]);
        return ones == 1;
    }
    // ceil(log2 v) for v >= 1
    int ceil_log2() const { return is_pow2() ? bit_length() - 1 : bit_length(); }
};

// col[n] = N(n,k) for n = 0..N, advanced from k to k+1 with
// N(n,k+1) = N(n-1,k+1) + N(n,k) + N(n-1,k)   (Sec. 2.4).
struct CountColumn {
    std::vector<BigU> col;
    int k = 0;
    explicit CountColumn(int N) : col(static_cast<size_t>(N) + 1, BigU(1u)) {}  // N(n,0) = 1
    bool advance() {
        std::vector<BigU> nxt(col.size());
        nxt[0] = BigU(0u);  // N(0,k>=1) = 0
        for (size_t n = 1; n < col.size(); ++n) {
            nxt[n] = nxt[n - 1];
            if (!nxt[n].add(col[n]) || !nxt[n].add(col[n - 1])) return false;
        }
        col.swap(nxt);
        ++k;
        return true;
    }
};

}  // namespace

static int index_bits_exact(int N, int K) {
    if (N < 1 || N > 4096 || K < 0 || K > 65535) return -1;
    CountColumn c(N);
    for (int k = 0; k < K; ++k)
        if (!c.advance()) return -1;
    return c.col[static_cast<size_t>(N)].ceil_log2();
}

int device_info(DeviceInfo* out) {
    static std::mutex mu;
    static std::map<int, DeviceInfo> memo;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find(dev);
    if (it == memo.end()) {
        DeviceInfo d;
        if ((e = cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return set_cuda_error(e);
        if ((e = cudaDeviceGetAttribute(&d.smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
            return set_cuda_error(e);
        d.smem_max -= 256;  // room for the kernels' few bytes of static shared memory (an mbarrier)
        it = memo.emplace(dev, d).first;
    }
    *out = it->second;
    return PVQ_OK;
}

int prepare_kernel(const void* kern, int threads, size_t smem, int* blocks_per_sm) {
    struct Key {
        const void* kern;
        int dev, threads;
        size_t smem;
        bool operator<(const Key& o) const {
            return std::tie(kern, dev, threads, smem) < std::tie(o.kern, o.dev, o.threads, o.smem);
        }
    };
    static std::mutex mu;
    static std::map<Key, int> memo;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    std::lock_guard<std::mutex> lock(mu);
    const Key key{kern, dev, threads, smem};
    auto it = memo.find(key);
    if (it == memo.end()) {
        // the attribute is per kernel and device: keep it at the largest size asked for so far
        size_t largest = smem;
        for (const auto& kv : memo)
            if (kv.first.kern == kern && kv.first.dev == dev) largest = std::max(largest, kv.first.smem);
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(largest))) !=
            cudaSuccess)
            return set_cuda_error(e);
        int per_sm = 0;
        if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem)) != cudaSuccess)
            return set_cuda_error(e);
        it = memo.emplace(key, per_sm).first;
    }
    *blocks_per_sm = it->second;
    return PVQ_OK;
}

// W for (N,K); memoised, since every hot call asks for it.
int code_words_for(int N, int K) {
    static std::mutex mu;
    static std::map<std::pair<int, int>, int> memo;
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find({N, K});
    if (it != memo.end()) return it->second;
    int bits = index_bits_exact(N, K);
    int W = bits < 0 ? 0 : std::max(1, (bits + 31) / 32);
    memo[{N, K}] = W;
    return W;
}

bool count_fills_its_words(int N, int K) {  // memoised like code_words_for: the count takes a while for large (N,K)
    static std::mutex mu;
    static std::map<std::pair<int, int>, bool> memo;
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find({N, K});
    if (it != memo.end()) return it->second;
    bool fills = false;
    if (N >= 1 && N <= 4096 && K >= 0 && K <= 65535) {
        CountColumn c(N);
        bool ok = true;
        for (int k = 0; k < K && ok; ++k) ok = c.advance();
        if (ok) {
            const BigU& v = c.col[static_cast<size_t>(N)];
            fills = v.is_pow2() && v.bit_length() > 32 && (v.bit_length() - 1) % 32 == 0;
        }
    }
    memo[{N, K}] = fills;
    return fills;
}

// The leading 24 bits of v >= 1 as the bits of an fp32 (what search_key computes on the device).
static uint32_t key_bits(const BigU& v) {
    const int e = v.bit_length() - 1;
    uint32_t mant = 0;  // bits e .. e-23 of v
    for (int b = 0; b < 24; ++b) {
        const int pos = e - b;
        const uint32_t bit = pos >= 0 ? (v.w[pos >> 5] >> (pos & 31)) & 1u : 0u;
        mant = (mant << 1) | bit;
    }
    return (static_cast<uint32_t>(e + 127) << 23) | (mant & 0x7fffffu);
}

// Layout of the search section (SearchLayout): the thresholds of every row are computed
// exactly, and each row gets the smallest number of key bits that puts every threshold in a
// bucket of its own.
const SearchLayout& search_layout_for(int N, int K) {
    static std::mutex mu;
    static std::map<std::pair<int, int>, SearchLayout> memo;
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find({N, K});
    if (it != memo.end()) return it->second;
    SearchLayout& S = memo[{N, K}];
    std::memset(&S, 0, sizeof S);
    int W = 0;
    {
        const int bits = index_bits_exact(N, K);
        W = bits < 0 ? 0 : std::max(1, (bits + 31) / 32);
    }
    if (W < 1 || W > 4 || K > 127 || K < 1 || N > kSearchMaxRows || N < 2) return S;
    // keys of T_n[m], m = 0..2K, n = 0..N-1
    const int M = 2 * K + 1;
    std::vector<uint32_t> keys(static_cast<size_t>(N) * M);
    std::vector<int> need(static_cast<size_t>(N));  // words that hold the row's largest threshold, N(n+1,K)
    {
        CountColumn c(N);  // col[n] = N(n,k)
        std::vector<BigU> V(static_cast<size_t>(N)), Vprev(static_cast<size_t>(N));
        for (int k = 0; k <= K; ++k) {
            if (k > 0 && !c.advance()) return S;
            for (int n = 0; n < N; ++n) {
                Vprev[n] = V[n];
                V[n].add(c.col[static_cast<size_t>(n)]);
                BigU u = V[n], v2 = V[n];
                u.add(Vprev[n]);
                v2.add(V[n]);
                keys[static_cast<size_t>(n) * M + 2 * k] = key_bits(u);
                if (k < K) keys[static_cast<size_t>(n) * M + 2 * k + 1] = key_bits(v2);
                if (k == K) need[n] = std::max(1, (u.bit_length() + 31) / 32);
            }
        }
        // N(N,K) = U(N-1,K) must stay below 2^(32 W): q = N(N,K) - code is computed in W words
        BigU top = V[N - 1];
        top.add(Vprev[N - 1]);
        if (top.bit_length() > 32 * W) return S;
    }
    const uint32_t key_one = 0x3f800000u;
    uint32_t boff = 0;
    for (int n = 0; n < N; ++n) {
        const uint32_t* kr = keys.data() + static_cast<size_t>(n) * M;
        const int last = n == 0 ? 1 : M - 1;  // row 0 (no dimension left) has the thresholds 1 and 2 only
        int sh = -1;
        for (int f = 0; f <= 23 && sh < 0; ++f) {
            const int s = 23 - f;
            bool distinct = true;
            for (int m = 1; m <= last && distinct; ++m) distinct = (kr[m] >> s) != (kr[m - 1] >> s);
            if (distinct) sh = s;
        }
        if (sh < 1) return S;  // the low key bits have to leave a bucket entry's low byte free
        S.rows.shift[n] = static_cast<uint8_t>(sh);
        S.rows.b_off[n] = boff;
        S.rows.b_len[n] = (kr[last] >> sh) - (key_one >> sh) + 1u;
        boff += S.rows.b_len[n];
    }
    if (N % 4 != 0) return S;
    S.plane = search_plane_of(K);
    uint32_t teoff = 0;
    for (int n = N - 1; n >= 0; --n) {  // a block of four rows takes the width of its top row
        const int w = need[static_cast<size_t>(n | 3)];
        S.rows.words[n] = static_cast<uint8_t>(w);
        S.count[w] += 1;
        S.rows.te_off[n] = teoff;
        teoff += static_cast<uint32_t>(S.plane) * w * 4u;
    }
    S.rec_off = kSearchHeader;
    S.b_off = S.rec_off + static_cast<uint32_t>(N) * 16u;
    S.t_off = (S.b_off + 4u * boff + 15u) & ~15u;
    S.te_bytes = (teoff + 15u) & ~15u;
    S.e_off = S.t_off + S.te_bytes;
    S.total = (S.e_off + S.te_bytes + 127u) & ~127u;
    if (S.total > kSearchLimit) return S;
    S.off = (table_layout(N, K, W).total + 127u) & ~127u;
    S.present = true;
    return S;
}

}  // namespace pvq

using namespace pvq;

// -------------------------------------------------------------- public: misc

extern "C" const char* pvq_strerror(int status) {
    switch (status) {
        case PVQ_OK: return "PVQ_OK";
        case PVQ_ERR_INVALID_ARG: return "PVQ_ERR_INVALID_ARG: bad pointer, size or parameter";
        case PVQ_ERR_UNSUPPORTED: return "PVQ_ERR_UNSUPPORTED: no kernel for this (N, K, G)";
        case PVQ_ERR_ALIGNMENT: return "PVQ_ERR_ALIGNMENT: pointer or leading dimension not aligned";
        case PVQ_ERR_TABLE_TOO_SMALL: return "PVQ_ERR_TABLE_TOO_SMALL: buffer smaller than required";
        case PVQ_ERR_CUDA: return "PVQ_ERR_CUDA: a CUDA call failed (pvq_last_cuda_error)";
        default: return "unknown pvq status";
    }
}

extern "C" int pvq_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" int pvq_index_bits(int N, int K, int* bits_out) {
    if (!bits_out) return PVQ_ERR_INVALID_ARG;
    int b = index_bits_exact(N, K);
    if (b < 0) return PVQ_ERR_INVALID_ARG;
    *bits_out = b;
    return PVQ_OK;
}

extern "C" int pvq_max_pulses(int N, int index_bits, int* K_out) {
    if (!K_out || N < 1 || N > 4096 || index_bits < 1 || index_bits > 32 * (kLimbs - 2))
        return PVQ_ERR_INVALID_ARG;
    CountColumn c(N);
    int K = 0;
    for (;;) {
        if (!c.advance()) break;
        const BigU& v = c.col[static_cast<size_t>(N)];
        // v <= 2^index_bits  <=>  bit_length <= index_bits, or v == 2^index_bits exactly
        int bl = v.bit_length();
        bool fits = bl <= index_bits || (bl == index_bits + 1 && v.is_pow2());
        if (!fits) break;
        K = c.k;
        if (K >= 65535) break;
    }
    *K_out = K;
    return PVQ_OK;
}

extern "C" int pvq_code_words(int N, int K, int* W_out) {
    if (!W_out) return PVQ_ERR_INVALID_ARG;
    int W = code_words_for(N, K);
    if (W == 0) return PVQ_ERR_INVALID_ARG;
    *W_out = W;
    return PVQ_OK;
}

extern "C" size_t pvq_count_table_bytes(int N, int K) {
    int W = code_words_for(N, K);
    if (W == 0 || N < 1 || K < 1) return 0;
    const SearchLayout& S = search_layout_for(N, K);
    return S.present ? static_cast<size_t>(S.off) + S.total : table_layout(N, K, W).total;
}

extern "C" size_t pvq_scale_row_stride(int64_t G, int scale_bits) {
    if (G < 1 || ((scale_bits < 1 || scale_bits > 8) && scale_bits != 16)) return 0;
    size_t bytes = static_cast<size_t>((G * scale_bits + 7) / 8);
    return (bytes + 3u) & ~static_cast<size_t>(3u);
}

// ------------------------------------------------------ status word of the encode-side calls

static thread_local uint32_t* g_encode_status = nullptr;

extern "C" int pvq_encode_status(uint32_t* d_status) {
    g_encode_status = d_status;
    return PVQ_OK;
}

// ------------------------------------------------------ bounds-checked build

static thread_local uint32_t* g_debug_status = nullptr;

#ifdef PVQ_DEBUG
namespace pvq {
// the global-table kernels are not part of the bounds-checked build
int launch_big(const BatchArgs&, int, int, int, bool, cudaStream_t) { return PVQ_ERR_UNSUPPORTED; }
}  // namespace pvq
#endif

extern "C" int pvq_debug_status(uint32_t* d_status) {
#ifdef PVQ_DEBUG
    g_debug_status = d_status;
    return PVQ_OK;
#else
    (void)d_status;
    return PVQ_ERR_UNSUPPORTED;
#endif
}

// ------------------------------------------------------ public: hot-path calls

namespace {

struct Common {
    int N, K, W, scale_bits;
};

int check_common(int N, int K, int scale_bits, const uint32_t* d_table, Common* out) {
    if (N < 2 || (N & (N - 1)) != 0 || K < 1) return PVQ_ERR_INVALID_ARG;
    if ((scale_bits < 1 || scale_bits > 8) && scale_bits != 16) return PVQ_ERR_INVALID_ARG;
    if (!d_table) return PVQ_ERR_INVALID_ARG;
    if (N < 8 || N > kMaxGroup || K > kMaxPulses) return PVQ_ERR_UNSUPPORTED;
    int W = code_words_for(N, K);
    if (W == 0) return PVQ_ERR_INVALID_ARG;
    if (W > kMaxWords) return PVQ_ERR_UNSUPPORTED;
    if (!is_aligned(d_table, 16)) return PVQ_ERR_ALIGNMENT;
    out->N = N;
    out->K = K;
    out->W = W;
    out->scale_bits = scale_bits;
    return PVQ_OK;
}

// Fills the geometry of one matrix; `need` says which pointers the call uses.
enum { NEED_X = 1, NEED_OUT = 2, NEED_CODES = 4, NEED_EDGES = 8, NEED_LEVELS = 16 };

int fill_matrix(const pvq_matrix_desc& d, int need, int dtype, const Common& c, MatrixArgs* m) {
    if (d.rows < 1 || d.cols < 1 || d.cols % c.N != 0) return PVQ_ERR_INVALID_ARG;
    const int64_t G = d.cols / c.N;
    if (G < 2) return PVQ_ERR_UNSUPPORTED;  // the quantile codebook needs two groups (beta > 0)
    if (G > 4096) return PVQ_ERR_UNSUPPORTED;  // groups per row (the encoders' row trees; see pvq.h)
    if (d.rows * G >= (int64_t(1) << 31)) return PVQ_ERR_UNSUPPORTED;
    if (need & NEED_X) {
        if (!d.d_x || d.ld < d.cols) return PVQ_ERR_INVALID_ARG;
        const int vec = dtype == PVQ_DTYPE_BF16 ? 8 : 4;
        if (!is_aligned(d.d_x, 16) || d.ld % vec != 0) return PVQ_ERR_ALIGNMENT;
    }
    if (need & NEED_OUT) {
        if (!d.d_out || d.ld_out < d.cols) return PVQ_ERR_INVALID_ARG;
        if (!is_aligned(d.d_out, 16) || d.ld_out % 8 != 0) return PVQ_ERR_ALIGNMENT;
    }
    if (need & NEED_CODES) {
        if (!d.d_codes || !d.d_scale_idx || !d.d_row_norm) return PVQ_ERR_INVALID_ARG;
        if (!is_aligned(d.d_codes, 4) || !is_aligned(d.d_scale_idx, 4) || !is_aligned(d.d_row_norm, 4))
            return PVQ_ERR_ALIGNMENT;
    }
    // the quantile codebook is not used with 16-bit amplitudes
    if ((need & NEED_EDGES) && c.scale_bits <= 8 && !d.d_edges) return PVQ_ERR_INVALID_ARG;
    if ((need & NEED_LEVELS) && c.scale_bits <= 8 && !d.d_levels) return PVQ_ERR_INVALID_ARG;
    m->x = d.d_x;
    m->out = d.d_out;
    m->codes = d.d_codes;
    m->scale_idx = d.d_scale_idx;
    m->row_norm = d.d_row_norm;
    m->edges = d.d_edges;
    m->levels = d.d_levels;
    m->rows = d.rows;
    m->cols = d.cols;
    m->ld = d.ld;
    m->ld_out = d.ld_out;
    m->G = static_cast<int>(G);
    m->sstride = static_cast<int>(pvq_scale_row_stride(G, c.scale_bits));
    m->rows_per_tile = 1;
    m->tile_begin = 0;
    return PVQ_OK;
}

int run_batch(const pvq_matrix_desc* descs, int count, int need, int dtype, int N, int K, int scale_bits,
              const uint32_t* d_table, uint32_t* d_status, int kind /*0 enc,1 dec,2 fused*/,
              pvq_stream_t stream, int rot_block = 0, const float* d_signs = nullptr, int amp_mode = 0) {
    if (!descs || count < 1 || count > kMaxBatch) return PVQ_ERR_INVALID_ARG;
    if (kind != 1 && dtype != PVQ_DTYPE_F32 && dtype != PVQ_DTYPE_BF16) return PVQ_ERR_INVALID_ARG;
    Common c;
    int st = check_common(N, K, scale_bits, d_table, &c);
    if (st != PVQ_OK) return st;
    BatchArgs a;
    std::memset(&a, 0, sizeof a);
    a.count = count;
    a.K = K;
    a.code_words = c.W;
    a.scale_bits = scale_bits;
    a.table = d_table;
    a.status = d_status;
    a.c_one = 1u;
    a.c_minus_one = 0xffffffffu;
    a.debug_status = g_debug_status;
    if (kind != 1 && !a.status) a.status = g_encode_status;  // the encode-side calls take no status argument
    if (amp_mode != 0 && amp_mode != 1) return PVQ_ERR_INVALID_ARG;
    a.amp_mode = amp_mode;
    if (rot_block != 0) {
        if (!d_signs || rot_block < N || (rot_block & (rot_block - 1)) != 0) return PVQ_ERR_INVALID_ARG;
        if (rot_block > 16384) return PVQ_ERR_UNSUPPORTED;
        for (int i = 0; i < count; ++i)
            if (descs[i].cols % rot_block != 0) return PVQ_ERR_INVALID_ARG;
        a.rot_block = rot_block;
        a.rot_signs = d_signs;
    }
    for (int i = 0; i < count; ++i) {
        st = fill_matrix(descs[i], need, dtype, c, &a.m[i]);
        if (st != PVQ_OK) return st;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // codes the shared-memory kernels are built for, by group size
    const int fast_words = c.N == 8 ? 2 : (c.N == 16 ? 3 : (c.N == 32 ? 4 : (c.N == 64 ? 6 : 0)));
    if (c.W > fast_words) {  // large groups, wide codes
        a.fused = kind == 2 ? 1 : 0;
        return launch_big(a, dtype, c.N, c.W, kind == 1, s);
    }
    if (kind == 1) return launch_decode(a, c.N, c.W, s);
    return launch_encode(a, dtype, c.N, c.W, kind == 2, s);
}

}  // namespace

extern "C" int pvq_encode(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                          int scale_bits, const uint32_t* d_table, const float* d_edges, uint32_t* d_codes,
                          uint8_t* d_scale_idx, float* d_row_norm, pvq_stream_t stream) {
    pvq_matrix_desc d;
    std::memset(&d, 0, sizeof d);
    d.d_x = d_x;
    d.d_codes = d_codes;
    d.d_scale_idx = d_scale_idx;
    d.d_row_norm = d_row_norm;
    d.d_edges = d_edges;
    d.rows = rows;
    d.cols = cols;
    d.ld = ld;
    return run_batch(&d, 1, NEED_X | NEED_CODES | NEED_EDGES, dtype, N, K, scale_bits, d_table, nullptr, 0,
                     stream);
}

extern "C" int pvq_decode(const uint32_t* d_codes, const uint8_t* d_scale_idx, const float* d_row_norm,
                          int64_t rows, int64_t cols, int N, int K, int scale_bits, const uint32_t* d_table,
                          const float* d_levels, void* d_out, int64_t ld_out, uint32_t* d_status,
                          pvq_stream_t stream) {
    pvq_matrix_desc d;
    std::memset(&d, 0, sizeof d);
    d.d_out = d_out;
    d.d_codes = const_cast<uint32_t*>(d_codes);
    d.d_scale_idx = const_cast<uint8_t*>(d_scale_idx);
    d.d_row_norm = const_cast<float*>(d_row_norm);
    d.d_levels = d_levels;
    d.rows = rows;
    d.cols = cols;
    d.ld_out = ld_out;
    return run_batch(&d, 1, NEED_OUT | NEED_CODES | NEED_LEVELS, PVQ_DTYPE_BF16, N, K, scale_bits, d_table,
                     d_status, 1, stream);
}

extern "C" int pvq_roundtrip(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                             int scale_bits, const uint32_t* d_table, const float* d_edges,
                             const float* d_levels, void* d_out, int64_t ld_out, pvq_stream_t stream) {
    pvq_matrix_desc d;
    std::memset(&d, 0, sizeof d);
    d.d_x = d_x;
    d.d_out = d_out;
    d.d_edges = d_edges;
    d.d_levels = d_levels;
    d.rows = rows;
    d.cols = cols;
    d.ld = ld;
    d.ld_out = ld_out;
    return run_batch(&d, 1, NEED_X | NEED_OUT | NEED_EDGES | NEED_LEVELS, dtype, N, K, scale_bits, d_table,
                     nullptr, 2, stream);
}

extern "C" int pvq_encode_batched(const pvq_matrix_desc* descs, int count, int dtype, int N, int K,
                                  int scale_bits, const uint32_t* d_table, pvq_stream_t stream) {
    return run_batch(descs, count, NEED_X | NEED_CODES | NEED_EDGES, dtype, N, K, scale_bits, d_table,
                     nullptr, 0, stream);
}

extern "C" int pvq_decode_batched(const pvq_matrix_desc* descs, int count, int N, int K, int scale_bits,
                                  const uint32_t* d_table, uint32_t* d_status, pvq_stream_t stream) {
    return run_batch(descs, count, NEED_OUT | NEED_CODES | NEED_LEVELS, PVQ_DTYPE_BF16, N, K, scale_bits,
                     d_table, d_status, 1, stream);
}

extern "C" int pvq_rotate_encode(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int block,
                                 const float* d_signs, int N, int K, int scale_bits, const uint32_t* d_table,
                                 const float* d_edges, uint32_t* d_codes, uint8_t* d_scale_idx,
                                 float* d_row_norm, pvq_stream_t stream) {
    if (block == 0) return PVQ_ERR_INVALID_ARG;
    pvq_matrix_desc d;
    std::memset(&d, 0, sizeof d);
    d.d_x = d_x;
    d.d_codes = d_codes;
    d.d_scale_idx = d_scale_idx;
    d.d_row_norm = d_row_norm;
    d.d_edges = d_edges;
    d.rows = rows;
    d.cols = cols;
    d.ld = ld;
    return run_batch(&d, 1, NEED_X | NEED_CODES | NEED_EDGES, dtype, N, K, scale_bits, d_table, nullptr, 0,
                     stream, block, d_signs);
}

extern "C" int pvq_rotate_roundtrip(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int block,
                                    const float* d_signs, int N, int K, int scale_bits,
                                    const uint32_t* d_table, const float* d_edges, const float* d_levels,
                                    void* d_out, int64_t ld_out, pvq_stream_t stream) {
    if (block == 0) return PVQ_ERR_INVALID_ARG;
    pvq_matrix_desc d;
    std::memset(&d, 0, sizeof d);
    d.d_x = d_x;
    d.d_out = d_out;
    d.d_edges = d_edges;
    d.d_levels = d_levels;
    d.rows = rows;
    d.cols = cols;
    d.ld = ld;
    d.ld_out = ld_out;
    return run_batch(&d, 1, NEED_X | NEED_OUT | NEED_EDGES | NEED_LEVELS, dtype, N, K, scale_bits, d_table,
                     nullptr, 2, stream, block, d_signs);
}

extern "C" int pvq_encode_amp(const void* d_x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                              int scale_bits, int amp_mode, const uint32_t* d_table, const float* d_edges,
                              uint32_t* d_codes, uint8_t* d_scale_idx, float* d_row_norm, pvq_stream_t stream) {
    pvq_matrix_desc d;
    std::memset(&d, 0, sizeof d);
    d.d_x = d_x;
    d.d_codes = d_codes;
    d.d_scale_idx = d_scale_idx;
    d.d_row_norm = d_row_norm;
    d.d_edges = d_edges;
    d.rows = rows;
    d.cols = cols;
    d.ld = ld;
    return run_batch(&d, 1, NEED_X | NEED_CODES | NEED_EDGES, dtype, N, K, scale_bits, d_table, nullptr, 0,
                     stream, 0, nullptr, amp_mode);
}
