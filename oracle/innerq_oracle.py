"""Plain CPU oracle for the InnerQ decode path.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import
this module; the CUDA library never does, and this module imports nothing from it.
It is written to be checked against the paper by eye: numpy, one step per line, no
blocking, no fusion.  Attention arithmetic is float64.  The quantiser's arithmetic is
float32/float16 where that rounding is part of the stored format (scales and
zero-points are fp16, Table "bits"), spelled out as single correctly-rounded IEEE
operations so that any other implementation can reproduce the stored bits.

What each function follows
  quantize_groups   Section "Asymmetric and Symmetric Quantization" (quant/dequant
                    equations, scale and zero-point definitions) and Section
                    "Hybrid Quantization" (per-group mask M chosen by the lower
                    reconstruction error, M kept in the scale's sign bit,
                    zero-point 0 when M = 0; Figure "hybrid").
  dequantize_groups hybrid dequantisation equation  S*K^ + M*Z.
  channel_norm      Section "Per-channel Normalization of K".
  OracleCache       Section "High-precision Window" (sink / recent windows, eviction
                    of the oldest recent tokens), Section "InnerQ" (K grouped per token
                    along channels, V grouped per channel along tokens), Section
                    "Latency" (one key token quantised per step, G value tokens every
                    G steps; the outer-grouped method does the reverse).
  dense_attention   the three attention equations S = QK^T, P = softmax(S/sqrt(d_h)),
                    O = PV, for one query token.

Readings taken where the paper is silent or inconsistent (each also listed in the
design notes of the repository):
  * Symmetric mode.  The text says "the asymmetric equations with Z = 0" (clip to
    [0, 2^b-1]) with S = max|G| / (2^b-1), and also says the codes are signed.  Both
    cannot hold.  Two variants are implemented: FULLRANGE (default) uses the
    symmetric integer range [-(2^(b-1)-1), 2^(b-1)-1] with S = max|G| / (2^(b-1)-1), so
    nothing is clipped and |x - x^| <= S/2; PAPER_LITERAL uses S = max|G| / (2^b-1) as
    printed with the signed b-bit range [-2^(b-1), 2^(b-1)-1], which clips the tails.
  * Rounding is round-half-to-even.  Codes are computed with the stored (fp16-rounded)
    scale and zero-point, as  rint((x - z) * (1/s)).
  * "Lower reconstruction error" = sum of absolute errors (the figure draws |G - G~|);
    a tie goes to symmetric.
  * Signed symmetric codes q are stored offset-binary, u = q + 2^(b-1), so one decoder
    x^ = s*u + z_eff serves all modes (z_eff = Z if M else -s*2^(b-1)).
  * norm_k = sqrt(max |K[:, k]|) is taken per (batch, KV head, channel) over all prefill
    tokens, fixed afterwards; a zero maximum gives norm 1.  Window tokens stay raw
    fp16; normalisation is applied when a key token is quantised, and folded into q
    (q' = q * norm) for the quantised rows only.
  * Value tokens are quantised G at a time; at prefill the first floor(n_mid/G)*G
    middle tokens are quantised and the remainder stays fp16 in front of the recent
    window.

Parity unpinned: how close the quantised result is to unquantised attention on real
models is only reported by the paper as task scores; nothing here pins it.
"""
from __future__ import annotations

import numpy as np

SYM, ASYM, HYBRID = 0, 1, 2
FULLRANGE, PAPER_LITERAL = 0, 1
INNER, OUTER, FP16 = 0, 1, 2

f32 = np.float32
f64 = np.float64


def sym_range(bits: int, sym_variant: int):
    """(denominator of the scale, lowest signed code, highest signed code)."""
    if sym_variant == FULLRANGE:
        den = 2 ** (bits - 1) - 1
        return den, -den, den
    return 2 ** bits - 1, -(2 ** (bits - 1)), 2 ** (bits - 1) - 1


def quantize_groups(x, bits: int, mode: int, sym_variant: int = FULLRANGE):
    """Quantise groups of values.  x: float32 [..., G]; every trailing row is one group.

    Returns a dict: code uint8 [..., G] (unsigned; offset-binary for symmetric groups),
    scale_bits uint16 [...] (fp16 scale, bit 15 = M), zero_bits uint16 [...] (fp16 Z if
    M else 0), flag bool [...], err_asym / err_sym float64 [...] (sum |x - x^|), and
    alt_code / alt_scale_bits / alt_zero_bits: the stored form of the candidate that was
    NOT chosen (what a group holds if M takes the other value; Figure "hybrid" computes
    both candidates and the mask selects one).  Tests compare against it the groups whose
    two errors are so close that float32 summation may order them the other way.
    """
    x = np.asarray(x, dtype=f32)
    L = 2 ** bits - 1
    half = 2 ** (bits - 1)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        # asymmetric candidate: Z = min(G), S = (max(G) - Z) / (2^b - 1)
        mn = x.min(axis=-1)
        mx = x.max(axis=-1)
        S_a = ((mx - mn) / f32(L)).astype(np.float16)
        Z = mn.astype(np.float16)
        s_a = S_a.astype(f32)[..., None]
        z = Z.astype(f32)[..., None]
        inv_a = f32(1.0) / s_a
        u_a = np.clip(np.rint((x - z) * inv_a), 0, L)
        u_a = np.where(s_a == 0, f32(0), u_a)
        # symmetric candidate: Z = 0, S = max|G| / den, signed codes
        den, q_lo, q_hi = sym_range(bits, sym_variant)
        am = np.abs(x).max(axis=-1)
        S_s = (am / f32(den)).astype(np.float16)
        s_s = S_s.astype(f32)[..., None]
        inv_s = f32(1.0) / s_s
        q_s = np.clip(np.rint(x * inv_s), q_lo, q_hi)
        q_s = np.where(s_s == 0, f32(0), q_s)
    # reconstruction errors against what a decoder will see (stored-precision S and Z)
    x64 = x.astype(f64)
    d_a = s_a.astype(f64) * u_a.astype(f64) + z.astype(f64)
    d_s = s_s.astype(f64) * q_s.astype(f64)
    e_a = np.abs(x64 - d_a).sum(axis=-1)
    e_s = np.abs(x64 - d_s).sum(axis=-1)
    if mode == SYM:
        flag = np.zeros(mn.shape, dtype=bool)
    elif mode == ASYM:
        flag = np.ones(mn.shape, dtype=bool)
    else:
        flag = e_a < e_s          # tie -> symmetric
    code_a, code_s = u_a.astype(np.uint8), (q_s + f32(half)).astype(np.uint8)
    scale_a, scale_s = (S_a.view(np.uint16) | np.uint16(0x8000)).astype(np.uint16), S_s.view(np.uint16)
    zero_a, zero_s = Z.view(np.uint16), np.zeros(mn.shape, dtype=np.uint16)
    pick = lambda m, a, s_: np.where(m, a, s_).astype(a.dtype)       # asymmetric candidate where m, else symmetric
    return dict(code=pick(flag[..., None], code_a, code_s), scale_bits=pick(flag, scale_a, scale_s),
                zero_bits=pick(flag, zero_a, zero_s), flag=flag, err_asym=e_a, err_sym=e_s,
                alt_code=pick(~flag[..., None], code_a, code_s), alt_scale_bits=pick(~flag, scale_a, scale_s),
                alt_zero_bits=pick(~flag, zero_a, zero_s))


def dequantize_groups(code, scale_bits, zero_bits, bits: int):
    """x^ = S*u + M*Z with offset-binary symmetric codes; float64 [..., G]."""
    scale_bits = np.asarray(scale_bits, dtype=np.uint16)
    zero_bits = np.asarray(zero_bits, dtype=np.uint16)
    flag = (scale_bits & 0x8000) != 0                      # test the bit: the scale may be -0.0
    s = (scale_bits & np.uint16(0x7FFF)).view(np.float16).astype(f64)
    Z = zero_bits.view(np.float16).astype(f64)
    z_eff = np.where(flag, Z, -s * (2 ** (bits - 1)))
    return s[..., None] * np.asarray(code).astype(f64) + z_eff[..., None]


def channel_norm(K, all_heads: bool = False):
    """norm[c] = sqrt(max_t |K[t, c]|) in float32, 0 -> 1.  K: fp16 [..., N, D] -> float32 [..., D].

    all_heads: the literal scope of the paper's formula, max over ALL leading axes (batch, heads) and tokens: one
    vector of D factors, broadcast back to every unit.  The default (the reading taken here, and the only one the
    CUDA path has) is one vector per (batch, KV head) unit."""
    m = np.abs(np.asarray(K).astype(f32)).max(axis=-2)
    if all_heads:
        m = np.broadcast_to(m.reshape(-1, m.shape[-1]).max(axis=0), m.shape)
    n = np.sqrt(m).astype(f32)
    return np.where(n == 0, f32(1.0), n).astype(f32)


def dense_attention(q, K, V, sm_scale=None):
    """Textbook single-query attention in float64.  q [D], K [N, D], V [N, D] -> [D]."""
    q = np.asarray(q, dtype=f64)
    K = np.asarray(K, dtype=f64)
    V = np.asarray(V, dtype=f64)
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(K.shape[-1])
    s = (K @ q) * sm_scale
    p = np.exp(s - s.max())
    p = p / p.sum()
    return p @ V


class _Store:
    """One quantised tensor (K or V) of all units: sink, quantised middle, fp16 recent.

    kind 'row'   : one token is one row; groups of G channels inside the token
                   (the paper's per-token group-wise quantisation); one token evicted per step.
    kind 'block' : groups of G tokens inside each channel (per-channel group-wise
                   quantisation); G tokens evicted every G steps.
    """

    def __init__(self, kind, U, D, G, bits, mode, sym_variant, w_sink, w_recent, cap):
        self.kind, self.U, self.D, self.G = kind, U, D, G
        self.bits, self.mode, self.sym_variant = bits, mode, sym_variant
        self.w_sink, self.w_recent = w_sink, w_recent
        self.sink = np.zeros((U, 0, D), dtype=np.float16)
        self.recent = np.zeros((U, 0, D), dtype=np.float16)
        self.n_q = 0
        self.code = np.zeros((U, cap, D), dtype=np.uint8)
        n_meta = (cap, D // G) if kind == "row" else (cap // G + 1, D)
        self.scale = np.zeros((U,) + n_meta, dtype=np.uint16)
        self.zero = np.zeros((U,) + n_meta, dtype=np.uint16)
        self.err_asym = np.zeros((U,) + n_meta, dtype=f64)
        self.err_sym = np.zeros((U,) + n_meta, dtype=f64)
        # the candidate that was not chosen, in stored form (only tests read it)
        self.alt_code = np.zeros((U, cap, D), dtype=np.uint8)
        self.alt_scale = np.zeros((U,) + n_meta, dtype=np.uint16)
        self.alt_zero = np.zeros((U,) + n_meta, dtype=np.uint16)

    # x: float32 [U, n, D] tokens to quantise (already normalised if K), n multiple of G for 'block'
    def _quantize_and_store(self, x):
        U, n, D = x.shape
        G = self.G
        if n == 0:
            return
        if self.kind == "row":
            r = quantize_groups(x.reshape(U, n, D // G, G), self.bits, self.mode, self.sym_variant)
            self.code[:, self.n_q:self.n_q + n] = r["code"].reshape(U, n, D)
            self.alt_code[:, self.n_q:self.n_q + n] = r["alt_code"].reshape(U, n, D)
            sl = slice(self.n_q, self.n_q + n)
        else:
            assert n % G == 0 and self.n_q % G == 0
            xg = x.reshape(U, n // G, G, D).transpose(0, 1, 3, 2)       # [U, groups, D, G]
            r = quantize_groups(xg, self.bits, self.mode, self.sym_variant)
            self.code[:, self.n_q:self.n_q + n] = r["code"].transpose(0, 1, 3, 2).reshape(U, n, D)
            self.alt_code[:, self.n_q:self.n_q + n] = r["alt_code"].transpose(0, 1, 3, 2).reshape(U, n, D)
            sl = slice(self.n_q // G, (self.n_q + n) // G)
        self.scale[:, sl] = r["scale_bits"]
        self.zero[:, sl] = r["zero_bits"]
        self.err_asym[:, sl] = r["err_asym"]
        self.err_sym[:, sl] = r["err_sym"]
        self.alt_scale[:, sl] = r["alt_scale_bits"]
        self.alt_zero[:, sl] = r["alt_zero_bits"]
        self.n_q += n

    def prefill(self, X, inv_norm):
        """X fp16 [U, N, D]; inv_norm float32 [U, D] or None."""
        U, N, D = X.shape
        ws, wr, G = self.w_sink, self.w_recent, self.G
        self.n_q = 0
        self.sink = X[:, :min(ws, N)].copy()
        n_mid = max(0, N - ws - wr)
        n_q = n_mid if self.kind == "row" else (n_mid // G) * G
        mid = X[:, ws:ws + n_q].astype(f32)
        if inv_norm is not None:
            mid = mid * inv_norm[:, None, :]
        self._quantize_and_store(mid)
        self.recent = X[:, min(N, ws + n_q):].copy()

    def append(self, x_new, n_total, inv_norm):
        """x_new fp16 [U, D]; n_total = token count including this token."""
        ws, wr, G = self.w_sink, self.w_recent, self.G
        if n_total <= ws:
            self.sink = np.concatenate([self.sink, x_new[:, None, :]], axis=1)
            return
        self.recent = np.concatenate([self.recent, x_new[:, None, :]], axis=1)
        n_ev = 0
        if self.kind == "row" and self.recent.shape[1] > wr:
            n_ev = 1
        if self.kind == "block" and self.recent.shape[1] == wr + G:
            n_ev = G
        if n_ev:
            ev = self.recent[:, :n_ev].astype(f32)
            if inv_norm is not None:
                ev = ev * inv_norm[:, None, :]
            self._quantize_and_store(ev)
            self.recent = self.recent[:, n_ev:].copy()

    def dequant(self, u):
        """float64 [n_q, D] reconstruction of unit u's quantised tokens (normalised domain for K)."""
        n, D, G = self.n_q, self.D, self.G
        if self.kind == "row":
            x = dequantize_groups(self.code[u, :n].reshape(n, D // G, G), self.scale[u, :n], self.zero[u, :n], self.bits)
            return x.reshape(n, D)
        code = self.code[u, :n].reshape(n // G, G, D).transpose(0, 2, 1)
        x = dequantize_groups(code, self.scale[u, :n // G], self.zero[u, :n // G], self.bits)
        return x.transpose(0, 2, 1).reshape(n, D)

    def n_meta(self):
        return self.n_q if self.kind == "row" else self.n_q // self.G


class OracleCache:
    """Quantised KV cache + decode attention for all (batch, KV head) units, on the host."""

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, group, k_bits, v_bits,
                 k_mode=HYBRID, v_mode=HYBRID, sym_variant=FULLRANGE, w_sink=4, w_recent=128,
                 grouping=INNER, k_normalize=1, sm_scale=0.0, norm_all_heads=False):
        assert n_q_heads % n_kv_heads == 0 and head_dim % group == 0
        self.B, self.Hq, self.Hkv, self.D = batch, n_q_heads, n_kv_heads, head_dim
        self.U = batch * n_kv_heads
        self.G, self.grouping = group, grouping
        self.w_sink, self.w_recent = w_sink, w_recent
        self.k_normalize = bool(k_normalize) and grouping == INNER
        self.norm_all_heads = bool(norm_all_heads)      # literal cross-head scope of the key norm (oracle only)
        self.sm_scale = float(sm_scale) if sm_scale else 1.0 / np.sqrt(head_dim)
        self.N = 0
        self.norm = np.ones((self.U, head_dim), dtype=f32)
        if grouping == FP16:
            self.K = np.zeros((self.U, 0, head_dim), dtype=np.float16)
            self.V = np.zeros((self.U, 0, head_dim), dtype=np.float16)
            return
        if grouping == OUTER:
            k_mode = v_mode = ASYM
        k_kind, v_kind = ("row", "block") if grouping == INNER else ("block", "row")
        args = dict(U=self.U, D=head_dim, G=group, sym_variant=sym_variant, w_sink=w_sink, w_recent=w_recent,
                    cap=max_tokens)
        self.k = _Store(k_kind, bits=k_bits, mode=k_mode, **args)
        self.v = _Store(v_kind, bits=v_bits, mode=v_mode, **args)

    def _inv_norm(self):
        return (f32(1.0) / self.norm) if self.k_normalize else None

    def prefill(self, K, V, norm=None):
        """K, V fp16 [B, Hkv, N, D] (or [U, N, D]).  `norm` overrides the computed key norm (tests only)."""
        K = np.asarray(K).reshape(self.U, -1, self.D)
        V = np.asarray(V).reshape(self.U, -1, self.D)
        self.N = K.shape[1]
        if self.grouping == FP16:
            self.K, self.V = K.copy(), V.copy()
            return
        if self.k_normalize:
            self.norm = channel_norm(K, self.norm_all_heads) if norm is None else np.asarray(norm, dtype=f32).reshape(self.U, self.D)
        self.k.prefill(K, self._inv_norm())
        self.v.prefill(V, None)

    def append(self, k_new, v_new):
        """k_new, v_new fp16 [B, Hkv, D]: the decode step's own token joins the cache."""
        k_new = np.asarray(k_new).reshape(self.U, self.D)
        v_new = np.asarray(v_new).reshape(self.U, self.D)
        self.N += 1
        if self.grouping == FP16:
            self.K = np.concatenate([self.K, k_new[:, None]], axis=1)
            self.V = np.concatenate([self.V, v_new[:, None]], axis=1)
            return
        self.k.append(k_new, self.N, self._inv_norm())
        self.v.append(v_new, self.N, None)

    def materialize(self, u):
        """(K~, V~) float64 [N, D]: what attention effectively sees for unit u, in the raw key domain."""
        if self.grouping == FP16:
            return self.K[u].astype(f64), self.V[u].astype(f64)
        kq = self.k.dequant(u)
        if self.k_normalize:
            kq = kq * self.norm[u].astype(f64)[None, :]
        Kt = np.concatenate([self.k.sink[u].astype(f64), kq, self.k.recent[u].astype(f64)], axis=0)
        Vt = np.concatenate([self.v.sink[u].astype(f64), self.v.dequant(u), self.v.recent[u].astype(f64)], axis=0)
        return Kt, Vt

    def decode(self, q, units=None, return_probs=False, n_hidden=0):
        """q fp16 [B, Hq, D] -> float64 [B, Hq, D].  Query head j reads KV head j // (Hq/Hkv).

        Scores: raw q against the fp16 windows, q' = q * norm against the dequantised
        (normalised) key rows; softmax over all N tokens; values from V's own partition.
        `units` restricts the work to some (batch, KV head) units (other rows stay NaN).
        `n_hidden` > 0 leaves the newest n_hidden tokens of the cache out (causal mask of a query that is
        n_hidden positions before the newest token; not in the paper, which decodes one token at a time).
        """
        n_vis = self.N - int(n_hidden)
        assert 0 < n_vis <= self.N
        q = np.asarray(q).reshape(self.B, self.Hq, self.D).astype(f64)
        r = self.Hq // self.Hkv
        out = np.full((self.B, self.Hq, self.D), np.nan, dtype=f64)
        probs = {}
        for u in (range(self.U) if units is None else units):
            b, h = divmod(u, self.Hkv)
            if self.grouping == FP16:
                Kt, Vt = self.materialize(u)
                for j in range(h * r, (h + 1) * r):
                    out[b, j] = dense_attention(q[b, j], Kt[:n_vis], Vt[:n_vis], self.sm_scale)
                continue
            k_sink, k_rec = self.k.sink[u].astype(f64), self.k.recent[u].astype(f64)
            k_hat = self.k.dequant(u)
            Vt = np.concatenate([self.v.sink[u].astype(f64), self.v.dequant(u), self.v.recent[u].astype(f64)], axis=0)
            norm = self.norm[u].astype(f64)
            for j in range(h * r, (h + 1) * r):
                qj = q[b, j]
                qn = qj * norm if self.k_normalize else qj
                d = np.concatenate([k_sink @ qj, k_hat @ qn, k_rec @ qj])[:n_vis]      # tokens oldest first
                s = d * self.sm_scale
                p = np.exp(s - s.max())
                p = p / p.sum()
                out[b, j] = p @ Vt[:n_vis]
                if return_probs:
                    probs[(b, j)] = p
        return (out, probs) if return_probs else out

    def decode_multi(self, q, units=None):
        """q fp16 [B, n_q, Hq, D] -> float64 [B, n_q, Hq, D]: n_q consecutive query tokens whose own keys and
        values are the newest n_q tokens of the cache; query i attends causally to tokens 0 .. N - n_q + i.
        (Verification step of speculative decoding; the paper itself decodes one token per step, Section
        "Preliminaries", so this is that definition applied n_q times to one cache state.)"""
        q = np.asarray(q)
        n_q = q.shape[1]
        out = np.empty((self.B, n_q, self.Hq, self.D), dtype=f64)
        for i in range(n_q):
            out[:, i] = self.decode(q[:, i], units=units, n_hidden=n_q - 1 - i)
        return out

    def export(self):
        """Canonical (unpacked) cache contents, tokens oldest first."""
        if self.grouping == FP16:
            return dict(n_tokens=self.N, K=self.K, V=self.V)
        k, v = self.k, self.v
        return dict(
            n_tokens=self.N, norm=self.norm.copy(),
            n_sink=k.sink.shape[1], n_qk=k.n_q, n_qv=v.n_q,
            n_k_recent=k.recent.shape[1], n_v_recent=v.recent.shape[1],
            k_sink=k.sink, v_sink=v.sink, k_recent=k.recent, v_recent=v.recent,
            k_code=k.code[:, :k.n_q], k_scale=k.scale[:, :k.n_meta()], k_zero=k.zero[:, :k.n_meta()],
            v_code=v.code[:, :v.n_q], v_scale=v.scale[:, :v.n_meta()], v_zero=v.zero[:, :v.n_meta()],
            k_err_asym=k.err_asym[:, :k.n_meta()], k_err_sym=k.err_sym[:, :k.n_meta()],
            v_err_asym=v.err_asym[:, :v.n_meta()], v_err_sym=v.err_sym[:, :v.n_meta()],
            k_alt_code=k.alt_code[:, :k.n_q], k_alt_scale=k.alt_scale[:, :k.n_meta()], k_alt_zero=k.alt_zero[:, :k.n_meta()],
            v_alt_code=v.alt_code[:, :v.n_q], v_alt_scale=v.alt_scale[:, :v.n_meta()], v_alt_zero=v.alt_zero[:, :v.n_meta()],
        )


def from_workload(w, max_tokens=None):
    """Build an OracleCache from any object with the workload attribute names (duck-typed)."""
    return OracleCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim,
                       max_tokens if max_tokens is not None else w.n_tokens + 1024,
                       w.group, w.k_bits, w.v_bits, w.k_mode, w.v_mode, w.sym_variant,
                       w.w_sink, w.w_recent, w.grouping, w.k_normalize)
