"""CPU checker for MixAttention's inference attention path (TEST INFRASTRUCTURE).

This file is test infrastructure, not part of the product: only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no
code with the CUDA library and never calls it.

What it computes (paper, Section 3, with Section 1 for causality and the KV
cache):

* a standard attention layer: the query at position i attends to every key
  j <= i;
* a sliding-window layer with window s: the query attends to the last s keys,
  the current token included, i.e. keys j with i - s < j <= i, and its cache
  only has to hold the past s tokens;
* KV-cache reuse: a layer may read the cache computed by an earlier layer and
  then has no cache of its own;
* grouped-query attention: query head h reads KV head h // (Hq / Hkv).

The method reaches exactly the textbook softmax-attention result, so the
"logical half" below is that definition written out in float64 over complete,
never-evicted K/V histories.  The "physical half" is an integer simulation of
a paged cache (16-token pages, FIFO free list, one block table per sequence)
and of ring buffers (slot = position mod s); attention computed from what the
physical half still stores must equal the logical half.

Quantised KV storage (FP8 E4M3 elements with a shared power-of-two scale per
head vector) is a reading of this library, not the paper's: see the section on
it below and its pins in tests/test_oracle_fp8.py.

Pins (tests/test_oracle_pins.py): dense brute-force masked softmax on tiny
inputs, torch's scaled_dot_product_attention in float64 for the no-window
case, closed forms (constant V, zero Q, window 1), needle keys on both sides
of the window edge, ring-vs-slice and reader-vs-owner invariants, the 1/l
cache-size law.  The paper prints no numeric attention output, so no
published value exists to pin against: beyond those pins, parity is unpinned
by the paper.
"""
from __future__ import annotations

from collections import deque
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

FULL = 0
SLIDING = 1

# status codes mirrored by the library's C ABI (values are part of the interface)
OK = 0
ERR_INVALID_ARG = -1
ERR_INVALID_LAYOUT = -2
ERR_NOT_OWNER = -3
ERR_OUT_OF_PAGES = -4
ERR_EMPTY_CONTEXT = -5
ERR_BAD_SEQ = -6
ERR_UNSUPPORTED = -7


class OracleError(Exception):
    def __init__(self, code: int, msg: str = ""):
        super().__init__(f"{code}: {msg}")
        self.code = code


# --------------------------------------------------------------------------
# layout (Section 3: per-layer mix of standard / sliding-window / reuse)
# --------------------------------------------------------------------------

def validate_layout(layout: Sequence[Tuple[int, int, int]]) -> None:
    """A reader names an EARLIER layer that computes its own cache (Section 3,
    paragraph on KV cache reuse); kind and window of a reader equal its owner's."""
    if len(layout) == 0:
        raise OracleError(ERR_INVALID_LAYOUT, "no layers")
    for l, (kind, window, owner) in enumerate(layout):
        if kind not in (FULL, SLIDING):
            raise OracleError(ERR_INVALID_LAYOUT, f"layer {l}: kind")
        if kind == SLIDING and window < 1:
            raise OracleError(ERR_INVALID_LAYOUT, f"layer {l}: window")
        if not (0 <= owner <= l):
            raise OracleError(ERR_INVALID_LAYOUT, f"layer {l}: owner must be an earlier layer or itself")
        okind, owindow, oowner = layout[owner]
        if oowner != owner:
            raise OracleError(ERR_INVALID_LAYOUT, f"layer {l}: owner {owner} does not own a cache")
        if okind != kind:
            raise OracleError(ERR_INVALID_LAYOUT, f"layer {l}: kind differs from owner's")
        if kind == SLIDING and owindow != window:
            raise OracleError(ERR_INVALID_LAYOUT, f"layer {l}: window differs from owner's")


def key_range(kind: int, window: int, i: int) -> Tuple[int, int]:
    """Half-open range [lo, hi) of key positions seen by the query at position i.

    Standard layer: all keys up to and including i.  Sliding layer, window s:
    the last s of them (Section 3)."""
    hi = i + 1
    lo = 0 if kind == FULL else max(0, hi - window)
    return lo, hi


def rope_rotate(x, positions, theta: float) -> np.ndarray:
    """Rotary position embedding as defined by the RoFormer paper the method cites
    (Section 3, last paragraph: the models use rotary embeddings): channel pairs (2i, 2i+1) of a
    head vector at position m are rotated by the angle m * theta^(-2i/d).

    x [n, heads, d] (d even), positions [n] integers.  float64 throughout."""
    x = _as64(x)
    n, _, d = x.shape
    pos = np.asarray(positions, dtype=np.float64).reshape(n, 1, 1)
    i = np.arange(d // 2, dtype=np.float64).reshape(1, 1, d // 2)
    ang = pos * np.power(float(theta), -2.0 * i / d)
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * c - x[..., 1::2] * s
    out[..., 1::2] = x[..., 0::2] * s + x[..., 1::2] * c
    return out


# --------------------------------------------------------------------------
# quantised KV storage (Section 2, "KV Quantization": storing the cached keys and
# values at reduced precision shrinks the cache and the bytes moved per step; the
# paper names the technique as compatible and fixes no format)
#
# Reading taken here: every head vector (one token, one KV head; K and V apart) is
# stored as FP8 E4M3 elements with one shared power-of-two scale, the block-scaled
# layout of the OCP Microscaling formats with the head vector as the block:
#   * E4M3 (OCP 8-bit floating point): 1 sign, 4 exponent (bias 7), 3 mantissa bits;
#     exponent field 0 = subnormals m/8 * 2^-6; the largest finite value is 448
#     (S.1111.110); S.1111.111 is NaN and there is no infinity;
#   * shared exponent X = floor(log2(max |x|)) - 8 (8 = exponent of E4M3's largest
#     binade), clamped to [-127, 127]; an all-zero vector takes X = -127;
#   * element = round-to-nearest-even of x / 2^X onto the E4M3 grid, saturating at
#     +-448 (a scaled maximum in (448, 512) rounds down to 448).
# The division by 2^X is exact, so every quantisation decision is a function of exact
# values: a CUDA implementation must reproduce codes and exponents bit for bit.
# --------------------------------------------------------------------------

E4M3_MAX = 448.0
E4M3_EMAX = 8


def e4m3_decode(codes) -> np.ndarray:
    """Value of each 8-bit E4M3 code (float64), from the format definition."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    val = np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    val = np.where((c & 0x7F) == 0x7F, np.nan, val)
    return sign * val


def e4m3_encode(y) -> np.ndarray:
    """Round-to-nearest-even of finite float64 values onto the E4M3 grid, saturating at
    +-448; returns the 8-bit codes.  Written from the grid itself: in the binade
    [2^e, 2^(e+1)) with e >= -6 the spacing is 2^(e-3); below 2^-6 (subnormals) it is 2^-9."""
    y = np.asarray(y, dtype=np.float64)
    a = np.abs(y)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)
    step = np.exp2(e - 3.0)
    q = np.rint(a / step) * step            # rint rounds halves to even; a / step is exact
    q = np.minimum(q, E4M3_MAX)
    # encode the grid value q (rounding may have carried it into the next binade)
    e2 = np.floor(np.log2(np.where(q > 0, q, 1.0)))
    normal = q >= 2.0 ** -6
    E = np.where(normal, e2 + 7.0, 0.0)
    M = np.where(normal, q / np.exp2(e2) * 8.0 - 8.0, q / 2.0 ** -9)
    code = (E.astype(np.int64) << 3) | M.astype(np.int64)
    code = np.where(np.signbit(y), code | 0x80, code)
    return code.astype(np.uint8)


def quantize_kv(x) -> Tuple[np.ndarray, np.ndarray]:
    """x [n, heads, d] (K or V rows) -> (codes uint8 [n, heads, d], X int32 [n, heads])."""
    x = _as64(x)
    amax = np.abs(x).max(axis=-1)
    X = np.floor(np.log2(np.where(amax > 0, amax, 1.0))) - E4M3_EMAX
    X = np.where(amax > 0, X, -127.0)
    X = np.clip(X, -127.0, 127.0)
    codes = e4m3_encode(x / np.exp2(X)[..., None])
    return codes, X.astype(np.int32)


def dequantize_kv(codes, X) -> np.ndarray:
    """Values the quantised cache stands for: element * 2^X (float64, exact)."""
    return e4m3_decode(codes) * np.exp2(np.asarray(X, dtype=np.float64))[..., None]


def kv_roundtrip(x) -> np.ndarray:
    """dequantize_kv(quantize_kv(x)): what a layer reads back from a quantised cache."""
    return dequantize_kv(*quantize_kv(x))


# --------------------------------------------------------------------------
# logical half: attention by definition, float64
# --------------------------------------------------------------------------

def softmax_attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """q [D], K [n, D], V [n, D] -> softmax(scale * K q) @ V, two-pass, float64."""
    s = scale * (K @ q)
    e = np.exp(s - s.max())
    p = e / e.sum()
    return p @ V


def _as64(x) -> np.ndarray:
    if hasattr(x, "detach"):           # torch tensor of any float dtype: exact widening
        x = x.detach().cpu().double().numpy()
    return np.asarray(x, dtype=np.float64)


def decode_attention(q, K_hist, V_hist, kind: int, window: int,
                     scale: Optional[float] = None, heads: Optional[Sequence[int]] = None) -> np.ndarray:
    """One decode step for one sequence and one layer.

    q [Hq, D]; K_hist, V_hist [n, Hkv, D] = the owner's complete history with
    the new token already appended; the query sits at position n-1.  Returns
    [Hq, D] (or [len(heads), D])."""
    q, K_hist, V_hist = _as64(q), _as64(K_hist), _as64(V_hist)
    n, n_kv, D = K_hist.shape
    n_q = q.shape[0]
    if n == 0:
        raise OracleError(ERR_EMPTY_CONTEXT, "no keys")
    G = n_q // n_kv
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    lo, hi = key_range(kind, window, n - 1)
    hs = range(n_q) if heads is None else heads
    out = np.empty((len(hs), D))
    for r, h in enumerate(hs):
        g = h // G
        out[r] = softmax_attend(q[h], K_hist[lo:hi, g], V_hist[lo:hi, g], scale)
    return out


def prefill_attention(q, K, V, kind: int, window: int, scale: Optional[float] = None,
                      rows: Optional[Sequence[int]] = None,
                      heads: Optional[Sequence[int]] = None,
                      prefix_len: int = 0) -> np.ndarray:
    """Prompt attention for one sequence.

    q [S, Hq, D] are the queries of positions prefix_len .. prefix_len + S - 1;
    K, V [prefix_len + S, Hkv, D] hold every key of the sequence up to the last
    query (the first prefix_len of them were cached by earlier calls).  Row i is
    the decode definition with the query at position prefix_len + i; with
    prefix_len = 0 the sequence starts at position 0.
    Returns [len(rows), len(heads), D]."""
    q, K, V = _as64(q), _as64(K), _as64(V)
    S, n_q, D = q.shape
    if K.shape[0] != prefix_len + S or V.shape[0] != prefix_len + S:
        raise OracleError(ERR_INVALID_ARG, "K, V must hold prefix_len + S keys")
    n_kv = K.shape[1]
    G = n_q // n_kv
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    rs = range(S) if rows is None else rows
    hs = range(n_q) if heads is None else heads
    out = np.empty((len(rs), len(hs), D))
    for a, i in enumerate(rs):
        lo, hi = key_range(kind, window, prefix_len + i)
        for c, h in enumerate(hs):
            g = h // G
            out[a, c] = softmax_attend(q[i, h], K[lo:hi, g], V[lo:hi, g], scale)
    return out


class LogicalCache:
    """Complete K/V history per (owner layer, sequence); never evicts."""

    def __init__(self, layout, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 scale: Optional[float] = None):
        validate_layout(layout)
        if n_q_heads % n_kv_heads:
            raise OracleError(ERR_INVALID_ARG, "Hq % Hkv")
        self.layout = list(layout)
        self.Hq, self.Hkv, self.D = n_q_heads, n_kv_heads, head_dim
        self.scale = 1.0 / np.sqrt(head_dim) if scale is None else scale
        self.hist: Dict[Tuple[int, int], List[np.ndarray]] = {}

    def append(self, layer: int, seq: int, K, V) -> None:
        kind, window, owner = self.layout[layer]
        if owner != layer:
            raise OracleError(ERR_NOT_OWNER, f"layer {layer} reuses layer {owner}'s cache")
        K, V = _as64(K), _as64(V)
        cur = self.hist.get((layer, seq))
        if cur is None:
            self.hist[(layer, seq)] = [K.copy(), V.copy()]
        else:
            cur[0] = np.concatenate([cur[0], K])
            cur[1] = np.concatenate([cur[1], V])

    def history(self, layer: int, seq: int):
        owner = self.layout[layer][2]
        cur = self.hist.get((owner, seq))
        if cur is None:
            z = np.zeros((0, self.Hkv, self.D))
            return z, z
        return cur[0], cur[1]

    def decode(self, layer: int, seq: int, q) -> np.ndarray:
        kind, window, _ = self.layout[layer]
        K, V = self.history(layer, seq)
        return decode_attention(q, K, V, kind, window, self.scale)

    def prefill(self, layer: int, seq: int, q, K, V) -> np.ndarray:
        """Attention over explicit prompt K/V (the owner's); an owner layer also
        records them.  The sequence must be empty (prompt starts at position 0)."""
        kind, window, owner = self.layout[layer]
        if owner == layer:
            if self.history(layer, seq)[0].shape[0] != 0:
                raise OracleError(ERR_UNSUPPORTED, "prefill into a non-empty cache")
            self.append(layer, seq, K, V)
        return prefill_attention(q, K, V, kind, window, self.scale)


# --------------------------------------------------------------------------
# physical half: paged full caches + ring buffers, integers only for indexing
# --------------------------------------------------------------------------

class PhysicalCache:
    """Integer simulation of the cache manager, plus storage addressed only
    through its indices.

    Rules (the paper leaves them open; this simulation fixes them):
    * one block table per sequence, shared by all full-attention owners; every
      full owner has a pool of n_pages pages indexed by the same page id;
    * free pages form a FIFO initialised from `free_order`; the page of logical
      block k = t // page_size is popped when the first token with that k is
      appended by any full owner, sequences in call order, tokens in position
      order; `seq_reset` pushes a sequence's pages back in logical-block order;
    * a sliding owner keeps a ring of `window` slots per sequence: token t
      lives in slot t mod window, so the ring holds the last min(len, window)
      tokens (Section 3: the cache stores the past s tokens);
    * each owner counts its own tokens per sequence; a reader uses its owner's.
    """

    def __init__(self, layout, n_kv_heads: int, head_dim: int, max_seqs: int,
                 n_pages: int, page_size: int = 16, free_order=None,
                 max_seq_len: int = 0, store_values: bool = True):
        validate_layout(layout)
        self.layout = list(layout)
        self.Hkv, self.D = n_kv_heads, head_dim
        self.max_seqs, self.n_pages, self.P = max_seqs, n_pages, page_size
        self.max_seq_len = max_seq_len if max_seq_len > 0 else n_pages * page_size
        self.max_blocks = -(-self.max_seq_len // page_size)
        order = list(range(n_pages)) if free_order is None else [int(x) for x in free_order]
        if sorted(order) != list(range(n_pages)):
            raise OracleError(ERR_INVALID_ARG, "free_order is not a permutation")
        self.free = deque(order)
        self.block_table: List[List[int]] = [[] for _ in range(max_seqs)]
        self.owners = [l for l, (_, _, o) in enumerate(self.layout) if o == l]
        self.full_owners = [l for l in self.owners if self.layout[l][0] == FULL]
        self.ring_owners = [l for l in self.owners if self.layout[l][0] == SLIDING]
        self.len = {o: [0] * max_seqs for o in self.owners}
        self.store_values = store_values
        self.pool: Dict[int, np.ndarray] = {}
        self.ring: Dict[int, np.ndarray] = {}
        if store_values:
            for o in self.full_owners:
                self.pool[o] = np.full((n_pages, page_size, 2, n_kv_heads, head_dim), np.nan)
            for o in self.ring_owners:
                W = self.layout[o][1]
                self.ring[o] = np.full((max_seqs, W, 2, n_kv_heads, head_dim), np.nan)

    # -- sizes -------------------------------------------------------------
    def cache_bytes(self, elem_bytes: int) -> int:
        """Bytes reserved for K/V storage: owners only; a reader adds nothing
        (Section 3: l layers sharing one cache shrink it by 1/l)."""
        per_tok = 2 * self.Hkv * self.D * elem_bytes
        total = len(self.full_owners) * self.n_pages * self.P * per_tok
        for o in self.ring_owners:
            total += self.max_seqs * self.layout[o][1] * per_tok
        return total

    # -- mutation ----------------------------------------------------------
    def _check_seq(self, seq: int) -> None:
        if not (0 <= seq < self.max_seqs):
            raise OracleError(ERR_BAD_SEQ, f"seq {seq}")

    def append(self, layer: int, seq_ids: Sequence[int], n_new: Optional[Sequence[int]] = None,
               K=None, V=None) -> None:
        """Append n_new[i] tokens to sequence seq_ids[i] of owner `layer`.
        K, V [sum n_new, Hkv, D] (None = indices only).  All or nothing."""
        if not (0 <= layer < len(self.layout)):
            raise OracleError(ERR_INVALID_ARG, "layer")
        kind, window, owner = self.layout[layer]
        if owner != layer:
            raise OracleError(ERR_NOT_OWNER, f"layer {layer}")
        n_new = [1] * len(seq_ids) if n_new is None else [int(x) for x in n_new]
        if len(set(seq_ids)) != len(seq_ids):
            raise OracleError(ERR_INVALID_ARG, "duplicate sequence in one call")
        need = 0
        for s, n in zip(seq_ids, n_new):
            self._check_seq(s)
            if n < 0:
                raise OracleError(ERR_INVALID_ARG, "n_new")
            end = self.len[layer][s] + n
            if end > self.max_seq_len:
                raise OracleError(ERR_INVALID_ARG, "max_seq_len")
            if kind == FULL:
                need += max(0, -(-end // self.P) - len(self.block_table[s]))
        if need > len(self.free):
            raise OracleError(ERR_OUT_OF_PAGES, f"need {need}, free {len(self.free)}")
        if K is not None:
            K, V = _as64(K), _as64(V)
        row = 0
        for s, n in zip(seq_ids, n_new):
            for _ in range(n):
                t = self.len[layer][s]
                if kind == FULL:
                    if t // self.P == len(self.block_table[s]):
                        self.block_table[s].append(self.free.popleft())
                    if self.store_values and K is not None:
                        page = self.block_table[s][t // self.P]
                        self.pool[layer][page, t % self.P, 0] = K[row]
                        self.pool[layer][page, t % self.P, 1] = V[row]
                else:
                    if self.store_values and K is not None:
                        self.ring[layer][s, t % window, 0] = K[row]
                        self.ring[layer][s, t % window, 1] = V[row]
                self.len[layer][s] = t + 1
                row += 1

    def seq_reset(self, seq: int) -> None:
        self._check_seq(seq)
        for o in self.owners:
            self.len[o][seq] = 0
        self.free.extend(self.block_table[seq])
        self.block_table[seq] = []

    # -- introspection (the bit-exact comparison surface) --------------------
    def get_len(self, layer: int, seq: int) -> int:
        self._check_seq(seq)
        return self.len[self.layout[layer][2]][seq]

    def get_block_table(self, seq: int) -> List[int]:
        self._check_seq(seq)
        return list(self.block_table[seq])

    def n_free_pages(self) -> int:
        return len(self.free)

    def get_ring_state(self, layer: int, seq: int) -> Tuple[int, int]:
        """(next_slot, n_valid) of the ring read by a sliding layer."""
        kind, window, owner = self.layout[layer]
        if kind != SLIDING:
            raise OracleError(ERR_INVALID_ARG, "not a sliding layer")
        n = self.get_len(layer, seq)
        return n % window, min(n, window)

    def locate(self, layer: int, seq: int, pos: int) -> Tuple[int, int]:
        """(page, slot) holding token `pos`: page id and offset in the page for
        a full layer, (-1, ring slot) for a sliding layer.  The token must
        still be stored."""
        kind, window, owner = self.layout[layer]
        n = self.get_len(layer, seq)
        lo = 0 if kind == FULL else max(0, n - window)
        if not (lo <= pos < n):
            raise OracleError(ERR_INVALID_ARG, "position not stored")
        if kind == FULL:
            return self.block_table[seq][pos // self.P], pos % self.P
        return -1, pos % window

    def read_kv(self, layer: int, seq: int, pos: int):
        page, slot = self.locate(layer, seq, pos)
        owner = self.layout[layer][2]
        if page >= 0:
            return self.pool[owner][page, slot, 0], self.pool[owner][page, slot, 1]
        return self.ring[owner][seq, slot, 0], self.ring[owner][seq, slot, 1]

    def gather(self, layer: int, seq: int):
        """K, V [m, Hkv, D] of every token the layer attends to, in storage
        order (ring order is physical, not chronological: softmax attention
        does not depend on the order of the keys)."""
        kind, window, owner = self.layout[layer]
        n = self.get_len(layer, seq)
        if kind == FULL:
            ks = [self.pool[owner][self.block_table[seq][t // self.P], t % self.P] for t in range(n)]
            kv = np.stack(ks) if ks else np.zeros((0, 2, self.Hkv, self.D))
        else:
            kv = self.ring[owner][seq, :min(n, window)]
        return kv[:, 0], kv[:, 1]

    def decode(self, layer: int, seq: int, q, scale: Optional[float] = None) -> np.ndarray:
        """Attention over what is physically stored (every stored key is in the
        layer's range by construction)."""
        K, V = self.gather(layer, seq)
        return decode_attention(q, K, V, FULL, 0, scale)
