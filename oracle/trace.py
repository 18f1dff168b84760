"""Tensor-lifetime trace of the chunked DiT block template (test infrastructure only).

The paper obtains lifetimes from one shape-only run of the pipeline and then
treats them as template-static ("Offline Static Layout"; Memory Analyzer).
There is no framework graph here, so the shape-only run is replaced by walking
the block's own op list: every op names what it reads and writes, a tensor is
born at the first op that writes it and dies after the last op that touches it
(half-open lifetime [birth, death), as in Algorithm 1's input).

Op order of one block with C sequence chunks (1 + 11 C ops):
    MOD
    for c: LN1A_c, KV_c, KROPE_c
    for c: LN1B_c, Q_c, QROPE_c, ATTN_c, PROJ_c
    for c: LN2_c, FFN1_c, FFN2_c
Chunk c covers token rows [floor(c S / C), floor((c+1) S / C)).

A phase may instead be split along the batch ("temporary serialization": only the planned steps
are split into sub-batches, which rejoin in the full-size tensors afterwards): piece c of C then
covers batch elements [floor(c B / C), floor((c+1) B / C)) and all S rows.

Sequence parallelism (the paper's SP: the latent sequence is split across GPUs; section
"Execution Configurations"): GPU p of P owns token rows [floor(p S / P), floor((p+1) S / P)).
Its trace has the same ops; every tensor holds only the owned rows -- chunks then cut the owned
rows, chunk c covering owned rows [floor(c n / C), floor((c+1) n / C)) of the n owned -- except
`kv`, which stays full-size: phase A fills the owned rows, the keys and values of the other GPUs
arrive in place (one all-gather) before phase B reads them.
"""
from __future__ import annotations

ALIGN = 256

KIND_INPUT, KIND_OUTPUT, KIND_FULL, KIND_CHUNK, KIND_WORKSPACE = range(5)
DTYPE_BF16, DTYPE_F32 = 0, 1

# row order of the tensor table; breaks ties between tensors born at the same op
_ROW = {n: i for i, n in enumerate(
    ("temb", "hid", "mod", "kv", "h1a", "h1b", "q", "o", "lse", "res", "h2", "g"))}


def align_up(n, a=ALIGN):
    return -(-n // a) * a


def chunk_rows(S, C):
    return [c * S // C for c in range(C + 1)]


class _Recorder:
    """Walks the op list; remembers first write and last touch of every tensor."""

    def __init__(self):
        self.t = 0
        self.tensors = {}

    def op(self, reads=(), writes=()):
        for name in reads:
            self.tensors[name]["death"] = self.t + 1
        for name, meta in writes:
            if name not in self.tensors:
                self.tensors[name] = dict(meta, name=name, birth=self.t)
            self.tensors[name]["death"] = self.t + 1
        self.t += 1


def phase_counts(chunks):
    """chunks: one count for all three phases, or a triple (C_A, C_B, C_C) for the key/value
    phase, the query/attention/projection phase and the feed-forward phase."""
    if isinstance(chunks, int):
        return (chunks, chunks, chunks)
    ca, cb, cc = (int(v) for v in chunks)
    return (ca, cb, cc)


SPLIT_ROWS, SPLIT_BATCH = 0, 1


def shard_rows(t, shard):
    """(first row, row count) owned by shard = (p, P); the whole sequence for shard None."""
    if shard is None:
        return 0, t.seq
    p, P = shard
    if P < 1 or not 0 <= p < P or P > t.seq:
        raise ValueError("shard must be (p, P) with 0 <= p < P <= S")
    r0 = p * t.seq // P
    return r0, (p + 1) * t.seq // P - r0


def piece_elems(t, C, axis, rows=None):
    """Token-row count times batch count of every piece of a phase split C ways along `axis`;
    `rows` = number of token rows the phase covers (all of them by default)."""
    rows = t.seq if rows is None else rows
    if axis == SPLIT_BATCH:
        b = chunk_rows(t.batch, C)
        return [(b[c + 1] - b[c]) * rows for c in range(C)]
    r = chunk_rows(rows, C)
    return [t.batch * (r[c + 1] - r[c]) for c in range(C)]


def trace(t, chunks, axes=(SPLIT_ROWS, SPLIT_ROWS, SPLIT_ROWS), shard=None):
    """Returns (tensors, n_ops).  tensors: list of dicts with name, kind, dtype, block,
    chunk, bytes (rounded up to 256), birth, death -- in id order (first birth, then
    table row).  `chunks` is an int or a per-phase triple (see phase_counts); with a triple
    the op list is MOD; C_A x (LN1A, KV, KROPE); C_B x (LN1B, Q, QROPE, ATTN, PROJ);
    C_C x (LN2, FFN1, FFN2) -- chunking applied only where the trace needs it.  `axes` says per
    phase whether its pieces are row chunks (all batch elements) or sub-batches (all rows).
    `shard` = (p, P): the trace of GPU p of P under sequence parallelism (see the module text)."""
    B, S, D, H, F, Dt = t.batch, t.seq, t.hidden, t.heads, t.ffn, t.temb_dim
    _, n_own = shard_rows(t, shard)
    CA, CB, CC = phase_counts(chunks)
    L = t.n_blocks
    for C, ax in zip((CA, CB, CC), axes):
        if ax not in (SPLIT_ROWS, SPLIT_BATCH):
            raise ValueError("axis must be 0 (rows) or 1 (batch)")
        if C < 1 or C > (B if ax == SPLIT_BATCH else n_own):
            raise ValueError("chunks must be in [1, rows] (rows) or [1, B] (batch)")
    eA, eB, eC = (piece_elems(t, C, ax, n_own) for C, ax in zip((CA, CB, CC), axes))
    rec = _Recorder()

    def meta(base, nbytes, kind, dtype, block, chunk=-1):
        return dict(base=base, bytes=align_up(nbytes), kind=kind, dtype=dtype, block=block, chunk=chunk)

    u = 2 * B * n_own * D                 # one bf16 hidden tensor over the owned rows
    u_all = 2 * B * S * D                 # ... over every row (keys and values of all GPUs)
    # inputs exist before the first op
    rec.tensors["temb"] = dict(meta("temb", 2 * B * Dt, KIND_INPUT, DTYPE_BF16, -1), name="temb", birth=0, death=1)
    rec.tensors["hid0"] = dict(meta("hid", u, KIND_INPUT, DTYPE_BF16, 0), name="hid0", birth=0, death=1)
    for l in range(L):
        hid, nxt = f"hid{l}", f"hid{l + 1}"
        mod, kv, res = f"mod{l}", f"kv{l}", f"res{l}"
        m_mod = (mod, meta("mod", 24 * B * D, KIND_FULL, DTYPE_F32, l))
        m_kv = (kv, meta("kv", 2 * u_all, KIND_FULL, DTYPE_BF16, l))
        m_res = (res, meta("res", 2 * u, KIND_FULL, DTYPE_F32, l))
        m_nxt = (nxt, meta("hid", u, KIND_OUTPUT if l + 1 == L else KIND_FULL, DTYPE_BF16, l + 1))
        rec.op(reads=["temb"], writes=[m_mod])                                   # MOD
        for c in range(CA):
            n = eA[c]
            h1a = (f"h1a{l}_{c}", meta("h1a", 2 * n * D, KIND_CHUNK, DTYPE_BF16, l, c))
            rec.op(reads=[hid, mod], writes=[h1a])                               # LN1A
            rec.op(reads=[h1a[0]], writes=[m_kv])                                # KV
            rec.op(reads=[kv], writes=[m_kv])                                    # KROPE (in place)
        for c in range(CB):
            n = eB[c]
            h1b = (f"h1b{l}_{c}", meta("h1b", 2 * n * D, KIND_CHUNK, DTYPE_BF16, l, c))
            q = (f"q{l}_{c}", meta("q", 2 * n * D, KIND_CHUNK, DTYPE_BF16, l, c))
            o = (f"o{l}_{c}", meta("o", 2 * n * D, KIND_CHUNK, DTYPE_BF16, l, c))
            lse = (f"lse{l}_{c}", meta("lse", 4 * H * n, KIND_CHUNK, DTYPE_F32, l, c))
            rec.op(reads=[hid, mod], writes=[h1b])                               # LN1B
            rec.op(reads=[h1b[0]], writes=[q])                                   # Q
            rec.op(reads=[q[0]], writes=[q])                                     # QROPE (in place)
            rec.op(reads=[q[0], kv], writes=[o, lse])                            # ATTN
            rec.op(reads=[o[0], hid, mod], writes=[m_res])                       # PROJ
        for c in range(CC):
            n = eC[c]
            h2 = (f"h2{l}_{c}", meta("h2", 2 * n * D, KIND_CHUNK, DTYPE_BF16, l, c))
            g = (f"g{l}_{c}", meta("g", 2 * n * F, KIND_CHUNK, DTYPE_BF16, l, c))
            rec.op(reads=[res, mod], writes=[h2])                                # LN2
            rec.op(reads=[h2[0]], writes=[g])                                    # FFN1
            rec.op(reads=[g[0], res, mod], writes=[m_nxt])                       # FFN2
    n_ops = rec.t
    rec.tensors[f"hid{L}"]["death"] = n_ops          # the output outlives the last op
    tensors = sorted(rec.tensors.values(), key=lambda d: (d["birth"], _ROW[d["base"]], d["chunk"]))
    for d in tensors:
        del d["base"]
    return tensors, n_ops
