"""Layout of the table blob, and what its search section has to hold, from the count table alone.

With V(n,k) = sum_{j<=k} N(n,j) (App. C.2) the thresholds of row n are
T_n[2k] = V(n,k) + V(n,k-1) and T_n[2k+1] = 2 V(n,k); the increment that goes with threshold m
is E_n[m] = T_{n-1}[2 (m >> 1)] - T_n[m] (T_{-1} = 0).  A row's bucket table maps the leading
bits of a value q to the number m0 of thresholds that lie in earlier buckets, and the row takes
the fewest leading bits for which no two of its thresholds share a bucket.  A bucket's entry is
m0 in its low byte and, above it, the key bits below the bucket number of the threshold that lies
in the bucket, left-aligned (all ones when the bucket has none); bit 8 marks a threshold below
2^24, which its key represents exactly.  Rows are stored in the
fewest 32-bit words that hold their largest threshold, classed in aligned blocks of four rows (a
block takes the width of its top row), and word plane by word plane: a row of w words is w planes
of `plane` words (64, 128 or 256, the first that holds 2K+2), plane j holding word j of every entry.  Plain Python
integers throughout; nothing here comes from the library.
"""


def blob_layout(N, K, W):
    """Byte offsets of the sections that follow the count table (see include/pvq.h)."""
    up = lambda v: (v + 127) & ~127
    rowlen = (K + 2) & ~1
    top = W if W <= 2 else (4 if W <= 4 else (6 if W <= 6 else (8 if W <= 8 else (12 if W <= 12 else (W + 3) & ~3))))
    bound_words = 16 if W <= 12 else 64
    off = up(N * (K + 1) * W * 4)
    lay = {"bound": off, "bound_words": bound_words, "rowlen": rowlen, "top": top}
    off += up(bound_words * 4)
    for name, words in (("walk_top", top), ("walk2", 2 if top > 2 else 0), ("walk1", 1 if top > 1 else 0)):
        lay[name] = (off, words)
        off += up(N * rowlen * words * 4)
    for name in ("enc_u", "enc_2v", "enc_v"):
        lay[name] = off
        off += up(N * (K + 2) * top * 4)
    lay["walkd"] = lay["start"] = lay["cenc0"] = lay["cenc1"] = None
    if N <= 64 and W <= 6:            # the sections of the shared-memory kernels
        lay["walkd"] = off
        off += up(N * rowlen * 8)
        lay["start"] = off
        off += 128
        crow = 32 if K + 1 <= 32 else (64 if K + 1 <= 64 else 128)
        cb = N * crow * top * 4
        if W <= 4 and K + 1 <= 128 and 2 * cb <= 160 * 1024:
            lay["cenc0"], lay["cenc1"], lay["crow"] = off, off + cb + 64, crow      # 64 bytes between the two
            off += 2 * cb + 128
    lay["total"] = off
    return lay


def key_bits(q):
    """q >= 1 truncated to its leading 24 bits, as the bits of an IEEE binary32."""
    e = q.bit_length() - 1
    mant = (q >> (e - 23)) if e >= 23 else (q << (23 - e))
    return ((e + 127) << 23) | (mant & 0x7FFFFF)


KEY_OF_ONE = 0x3F800000
LIMIT = 184 * 1024
MAGIC = 0x53515650


def thresholds(count, N, K):
    """T[n][m] for n = 0..N-1, m = 0..2K, from count[n][k] = N(n,k)."""
    T = []
    for n in range(N):
        V, acc = [0], 0
        for k in range(K + 1):
            acc += count[n][k]
            V.append(acc)               # V[k + 1] = V(n,k), V[0] = V(n,-1)
        row = []
        for k in range(K + 1):
            row.append(V[k + 1] + V[k])
            if k < K:
                row.append(2 * V[k + 1])
        T.append(row)
    return T


def section(count, N, K, W, blob_bytes_before):
    """None where the decoder walks; else the layout and contents of the section."""
    if not (1 <= W <= 4 and 1 <= K <= 127 and 2 <= N <= 64):
        return None
    T = thresholds(count, N, K)
    if T[N - 1][2 * K] >= 1 << (32 * W):       # N(N,K) = T_{N-1}[2K]
        return None
    if N % 4:
        return None
    need = [max(1, (T[n][2 * K].bit_length() + 31) // 32) for n in range(N)]
    words = [need[n | 3] for n in range(N)]
    plane = 64 if 2 * K + 2 <= 64 else (128 if 2 * K + 2 <= 128 else 256)
    te_offs, teoff = [0] * N, 0
    for n in range(N - 1, -1, -1):              # the widest rows come first
        te_offs[n] = teoff
        teoff += plane * words[n] * 4
    shifts, lens, offs, tables = [], [], [], []
    boff = 0
    for n in range(N):
        last = 1 if n == 0 else 2 * K
        keys = [key_bits(t) for t in T[n][:last + 1]]
        for f in range(24):
            sh = 23 - f
            ids = [k >> sh for k in keys]
            if all(a != b for a, b in zip(ids, ids[1:])):
                break
        else:
            return None
        if sh < 1:
            return None
        base = KEY_OF_ONE >> sh
        length = ids[-1] - base + 1
        tab = []
        for m, b in enumerate(ids):
            tab += [0xFFFFFF00 | m] * (b - base - len(tab))            # buckets without a threshold
            exact = 0x100 if T[n][m] < 1 << 24 else 0                  # equal keys are equal numbers there
            tab.append(((keys[m] << (32 - sh)) & 0xFFFFFFFF) | exact | m)  # the bucket of threshold m
        assert len(tab) == length
        shifts.append(sh)
        lens.append(length)
        offs.append(boff)
        tables.append(tab)
        boff += length
    rec_off = 32
    b_off = rec_off + 16 * N
    t_off = (b_off + 4 * boff + 15) & ~15
    te_bytes = (teoff + 15) & ~15
    e_off = t_off + te_bytes
    total = (e_off + te_bytes + 127) & ~127
    if total > LIMIT:
        return None
    E = []
    for n in range(N):
        row = []
        for m in range(2 * K + 1):
            nxt = T[n - 1][2 * (m >> 1)] if n >= 1 else 0
            row.append((nxt - T[n][m]) & ((1 << (32 * words[n])) - 1))
        E.append(row)
    return dict(off=(blob_bytes_before + 127) & ~127, words=words, plane=plane, te_offs=te_offs,
                counts=[words.count(w) for w in (4, 3, 2, 1)], rec_off=rec_off, b_off=b_off, t_off=t_off, e_off=e_off,
                te_bytes=te_bytes, total=total, shifts=shifts, lens=lens, offs=offs, tables=tables, T=T, E=E)


def decode_with(sec, count, code, N, K, ties=None):
    """The point of `code`, found the way the section is meant to be used; `ties` (a list) collects
    the positions where the key bits could not decide."""
    q = count[N][K] - code
    k, y = K, []
    for i in range(N):
        n = N - 1 - i
        sh = sec["shifts"][n]
        key = key_bits(q)
        entry = sec["tables"][n][(key >> sh) - (KEY_OF_ONE >> sh)]
        x = (key << (32 - sh)) & 0xFFFFFFFF
        m0 = entry & 0xFF
        m = m0 + (1 if x > entry else 0)
        if (entry - x) & 0xFFFFFFFF < 256:          # same leading 24 bits as the threshold: compare in full
            m = m0 + (1 if sec["T"][n][m0] < q else 0)
            if ties is not None:
                ties.append(i)
        assert sec["T"][n][m] >= q and (m == 0 or sec["T"][n][m - 1] < q)
        kp = m >> 1
        y.append(k - kp if m & 1 else kp - k)
        q += (sec["T"][n - 1][2 * kp] if n >= 1 else 0) - sec["T"][n][m]
        k = kp
    return y
