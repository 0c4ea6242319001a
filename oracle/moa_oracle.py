"""CPU oracle for the Mixture-of-Attentions drafter forward step (arXiv 2410.03804).

TEST INFRASTRUCTURE ONLY. Nothing on the product path may import this file;
only the tests, the smoke check and the CPU-baseline leg of the benchmark do.
It shares no code with the CUDA path and is deliberately plain and slow:
numpy in fp64, one step of the paper's method per function, in the paper's
order. numpy's matmul / sort serve as library primitives for single steps.

What the paper fixes and what is a reading of it
------------------------------------------------
The paper (Section 3.1, Algorithm 1, Section 2.2, hyper-parameter table in
Appendix A.1) fixes: LSA = bidirectional self-attention over the layer axis,
tokens independent, followed by a mean over layers; SA = causal self-attention
over token embeddings (tree-masked while drafting a tree); CA = unmasked
cross-attention from SA outputs into keys/values derived from the LSA output;
LM head + softmax; an EAGLE-2-style tree: expand the B most probable, rank the
B*B children by joint probability, keep B per level, D levels, finally keep the
m best of the B + (D-1)*B*B pool. Attention softmax is done in higher
precision than the storage type (Section 4, last paragraph before 4.1).

The paper is silent on normalisation, biases, activation, positional encoding
and block wiring. This oracle takes the Llama-style reading: pre-RMSNorm with a
learnable gain before every attention and MLP, no biases, SwiGLU MLP, residual
connections; rotary position embedding (half-split pairing) in SA only; none in
LSA or CA; the LLM's final RMSNorm gain precedes the LM head; the MLP listed
"after LSA" is applied per (token, layer) row before the mean. Joint
probabilities are sums of fp32 log-probabilities. Ties break towards the
smaller index everywhere.

Target Layer Inference (Section 3.2): with n_tli = N > 0 the N last LLM decoder layers run on every drafted
row between the CA block and the LM head, each over the LLM's own cache of that layer (positions <= t) plus
the keys / values of the row's drafted ancestors; a Llama decoder layer (pre-RMSNorm, rotary embedding, GQA,
SwiGLU, residuals) with weights "tli{l}_*", l = 0 the earliest of the N.

Storage precision: with store="bf16" every tensor that the method keeps in
the 16-bit storage type between two matrix products is rounded to bfloat16
(round to nearest even) at that point -- normalised activations entering a
projection, projected q / k / v, attention outputs, the gated MLP hidden
vector, cache entries and the reported LSA / drafter outputs; the residual
stream and all sums stay in full precision, as "16-bit storage, softmax and
accumulation in higher precision" (Section 4) implies. Top-B decisions are
compared in this mode, so that both sides decide in the same precision;
values are compared against the unrounded mode (store=None).

Parity status: every function below is pinned by tests/test_oracle_pins.py
against closed forms, library routines, brute force or invariants. The model's
outputs are NOT pinned against the authors' trained system (no worked example,
weights or code exist here): "parity unpinned" in that sense only.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# elementary steps
# --------------------------------------------------------------------------
def rmsnorm(x, g, eps):
    """n(x; g) = x * g / sqrt(mean(x^2) + eps), over the last axis."""
    x = np.asarray(x, F64)
    g = np.asarray(g, F64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * g / np.sqrt(ms + eps)


def softmax(a):
    """Softmax over the last axis: subtract the max, exponentiate, divide by the sum."""
    a = np.asarray(a, F64)
    e = np.exp(a - np.max(a, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def silu(x):
    x = np.asarray(x, F64)
    return x / (1.0 + np.exp(-x))


def linear(x, w):
    """y = W x for a row-major weight W[out, in]; x may carry leading row axes."""
    return np.matmul(np.asarray(x, F64), np.asarray(w, F64).T)


def swiglu_mlp(u, w_gate, w_up, w_down, rnd=lambda t: t):
    """W_down (silu(W_gate u) * (W_up u)); rnd rounds the gated hidden vector (a stored tensor)."""
    return linear(rnd(silu(linear(u, w_gate)) * linear(u, w_up)), w_down)


def attend(q, K, V):
    """Attention core for ONE query vector: softmax(q.K^T / sqrt(dh)) V.

    q [dh], K [n, dh], V [n, dh] -> [dh]."""
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    a = K @ q / np.sqrt(q.shape[-1])
    p = softmax(a)
    return p @ V


def kv_head_of(h, hq, hkv):
    """Grouped-query attention: query head h reads kv head h // (hq // hkv)."""
    return h // (hq // hkv)


def rope(x, pos, theta):
    """Rotary embedding of x [..., dh] at integer position pos.

    Element i (< dh/2) is paired with element i + dh/2 and the pair is rotated
    by the angle pos * theta^(-2i/dh). theta == 0 disables the rotation."""
    x = np.asarray(x, F64)
    if theta == 0:
        return x.copy()
    dh = x.shape[-1]
    half = dh // 2
    i = np.arange(half, dtype=F64)
    ang = float(pos) * theta ** (-2.0 * i / dh)
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def round_bf16(x):
    """Round to the nearest bfloat16 (ties to even), returned as float64."""
    x32 = np.ascontiguousarray(np.asarray(x, np.float32))
    bits = x32.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32).astype(F64).reshape(np.shape(x))


def lm_head_topk(o_hat, final_norm, w_lm, eps, B, rnd=lambda t: t):
    """LM head, log-softmax and the B most probable tokens (Eq. 1; Section 2.2).

    z = W_lm n(o_hat; g_final); logp = z - logsumexp(z).
    Order: log-probability descending, token id ascending on equality.
    Returns (ids [B] int64, logp [B] float64, z [V] float64)."""
    z = linear(rnd(rmsnorm(o_hat, final_norm, eps)), w_lm)
    zmax = np.max(z)
    lse = zmax + np.log(np.sum(np.exp(z - zmax)))
    logp = z - lse
    order = np.lexsort((np.arange(z.shape[0]), -logp))[:B]
    return order.astype(np.int64), logp[order], z


# --------------------------------------------------------------------------
# the drafter
# --------------------------------------------------------------------------
class Drafter:
    """The drafter's layers, one method per step of Algorithm 1.

    cfg: mapping with d_model, n_stack, d_stack, vocab, head_dim, lsa_hq,
    lsa_hkv, sa_hq, sa_hkv, ca_hq, ca_hkv, rms_eps, rope_theta.
    weights: mapping name -> array [out, in] (any float dtype; widened to fp64
    where used)."""

    def __init__(self, cfg, weights, cache_f64=True, store=None):
        self.c = dict(cfg)
        self.w_raw = weights
        self._cache = {} if cache_f64 else None
        assert store in (None, "bf16")
        self.rnd = round_bf16 if store == "bf16" else (lambda t: t)

    def w(self, name):
        if self._cache is None:
            return np.asarray(self.w_raw[name], F64)
        if name not in self._cache:
            self._cache[name] = np.asarray(self.w_raw[name], F64)
        return self._cache[name]

    # ---- Layer Self-Attention (Section 3.1.1, "Layer Self-Attention") -----
    def lsa_rows(self, X):
        """LSA block for ONE token, before the mean. X [S, D_in] -> Z [S, D_in].

        Rows of X are the S stacked layer activations; attention runs over
        these S rows with a full (bidirectional) mask and no positional term."""
        c = self.c
        S = X.shape[0]
        dh, hq, hkv = c["head_dim"], c["lsa_hq"], c["lsa_hkv"]
        X = np.asarray(X, F64)
        rnd = self.rnd
        U = rnd(rmsnorm(X, self.w("lsa_norm1"), c["rms_eps"]))
        Q = rnd(linear(U, self.w("lsa_wq"))).reshape(S, hq, dh)
        K = rnd(linear(U, self.w("lsa_wk"))).reshape(S, hkv, dh)
        V = rnd(linear(U, self.w("lsa_wv"))).reshape(S, hkv, dh)
        O = np.zeros((S, hq, dh), F64)
        for h in range(hq):
            g = kv_head_of(h, hq, hkv)
            for s in range(S):
                O[s, h] = attend(Q[s, h], K[:, g], V[:, g])
        Y = X + linear(rnd(O).reshape(S, hq * dh), self.w("lsa_wo"))
        Z = Y + self.mlp(rnd(rmsnorm(Y, self.w("lsa_norm2"), c["rms_eps"])), "lsa")
        return Z

    def mlp(self, u, block):
        """SwiGLU MLP of one block; the gated hidden vector is a stored tensor."""
        return swiglu_mlp(u, self.w(block + "_wgate"), self.w(block + "_wup"), self.w(block + "_wdown"), self.rnd)

    def lsa_token(self, X):
        """LSA followed by the mean aggregation over the layer axis: [S, D_in] -> [D_in]."""
        return np.mean(self.lsa_rows(X), axis=0)

    def lsa_forward(self, h_stack):
        """kv = LSA_layer_with_mean(h) (Algorithm 1, both LSA_layer_with_mean steps): every
        token independently. h_stack [n_tok, S, D_in] -> [n_tok, D_in]."""
        return np.stack([self.lsa_token(h_stack[t]) for t in range(h_stack.shape[0])]) \
            if h_stack.shape[0] else np.zeros((0, self.c["d_stack"]), F64)

    # ---- Cross-attention keys / values (Section 3.1.2, "Cross-Attention") -
    def ca_kv(self, kv):
        """K_c = W_k n(kv), V_c = W_v n(kv): one row per context position.
        kv [n, D_in] -> K_c, V_c [n, Hkv, dh]."""
        c = self.c
        u = self.rnd(rmsnorm(kv, self.w("ca_normkv"), c["rms_eps"]))
        n = u.shape[0]
        return (self.rnd(linear(u, self.w("ca_wk"))).reshape(n, c["ca_hkv"], c["head_dim"]),
                self.rnd(linear(u, self.w("ca_wv"))).reshape(n, c["ca_hkv"], c["head_dim"]))

    # ---- Self-attention (Section 3.1.2, "Self-Attention") -----------------
    def sa_qkv(self, tok, pos):
        """Embedding, pre-norm, q/k/v projections and rotation for one token
        at absolute position pos. Returns e [E], q [Hq,dh], k [Hkv,dh], v [Hkv,dh]."""
        c = self.c
        dh = c["head_dim"]
        e = np.asarray(self.w_raw["embed"][int(tok)], F64)
        u = self.rnd(rmsnorm(e, self.w("sa_norm1"), c["rms_eps"]))
        q = self.rnd(rope(linear(u, self.w("sa_wq")).reshape(c["sa_hq"], dh), pos, c["rope_theta"]))
        k = self.rnd(rope(linear(u, self.w("sa_wk")).reshape(c["sa_hkv"], dh), pos, c["rope_theta"]))
        v = self.rnd(linear(u, self.w("sa_wv")).reshape(c["sa_hkv"], dh))
        return e, q, k, v

    def sa_block(self, e, q, K, V):
        """SA block for one row, given its embedding e, rotated queries q
        [Hq,dh] and the key/value set it may see, K, V [n, Hkv, dh] (the row's
        own key and value included by the caller). Returns x [E]."""
        c = self.c
        hq, hkv, dh = c["sa_hq"], c["sa_hkv"], c["head_dim"]
        o = np.zeros((hq, dh), F64)
        for h in range(hq):
            g = kv_head_of(h, hq, hkv)
            o[h] = attend(q[h], K[:, g], V[:, g])
        a = e + linear(self.rnd(o).reshape(hq * dh), self.w("sa_wo"))
        return a + self.mlp(self.rnd(rmsnorm(a, self.w("sa_norm2"), c["rms_eps"])), "sa")

    # ---- Cross-attention block (Section 3.1.2; Algorithm 1, CA_layer step) -------
    def ca_block(self, x, K_c, V_c):
        """CA block for one row: queries from x, keys/values = ALL cached
        K_c, V_c [n, Hkv, dh]; no mask at generation time, no positional term."""
        c = self.c
        hq, hkv, dh = c["ca_hq"], c["ca_hkv"], c["head_dim"]
        qc = self.rnd(linear(self.rnd(rmsnorm(x, self.w("ca_normq"), c["rms_eps"])), self.w("ca_wq"))).reshape(hq, dh)
        o = np.zeros((hq, dh), F64)
        for h in range(hq):
            g = kv_head_of(h, hq, hkv)
            o[h] = attend(qc[h], K_c[:, g], V_c[:, g])
        cc = x + linear(self.rnd(o).reshape(hq * dh), self.w("ca_wo"))
        return cc + self.mlp(self.rnd(rmsnorm(cc, self.w("ca_norm2"), c["rms_eps"])), "ca")

    # ---- Target Layer Inference (Section 3.2): the last TLI frozen LLM decoder layers ----------
    def tli_layers(self):
        """Number of LLM decoder layers applied between the CA block and the LM head (TLI; 0 = none)."""
        return int(self.c.get("n_tli", 0))

    def tli_layer(self, l, x, pos, K, V):
        """One frozen LLM decoder layer f^l_decoder on one drafted row (Section 3.2, the second line of the
        drafter's equation; Algorithm 1, the loop over l): x [E] is o_hat^l, K, V [n, Hkv, dh] are the layer's
        cached keys / values the row may see (positions <= t from the LLM, then its drafted ancestors), the row's
        own key / value joins them. Llama-style reading as for the drafter's own blocks: pre-RMSNorm, rotary
        embedding at the row's absolute position, GQA, SwiGLU, residuals. Returns (o_hat^{l+1}, k, v)."""
        c = self.c
        dh, hq, hkv = c["head_dim"], c["tli_hq"], c["tli_hkv"]
        w = lambda n: self.w(f"tli{l}_{n}")
        x = np.asarray(x, F64)
        u = self.rnd(rmsnorm(x, w("norm1"), c["rms_eps"]))
        q = self.rnd(rope(linear(u, w("wq")).reshape(hq, dh), pos, c["rope_theta"]))
        k = self.rnd(rope(linear(u, w("wk")).reshape(hkv, dh), pos, c["rope_theta"]))
        v = self.rnd(linear(u, w("wv")).reshape(hkv, dh))
        Kf = np.concatenate([np.asarray(K, F64), k[None]], axis=0)
        Vf = np.concatenate([np.asarray(V, F64), v[None]], axis=0)
        o = np.zeros((hq, dh), F64)
        for h in range(hq):
            g = kv_head_of(h, hq, hkv)
            o[h] = attend(q[h], Kf[:, g], Vf[:, g])
        a = x + linear(self.rnd(o).reshape(hq * dh), w("wo"))
        out = a + swiglu_mlp(self.rnd(rmsnorm(a, w("norm2"), c["rms_eps"])), w("wgate"), w("wup"), w("wdown"), self.rnd)
        return out, k, v

    def head(self, o_hat, B):
        return lm_head_topk(o_hat, self.w("final_norm"), self.w("lm_head"), self.c["rms_eps"], B, self.rnd)

    # ---- prefix of the self-attention cache -------------------------------
    def sa_prefix(self, toks, start=0):
        """Rotated keys and values of prompt / accepted tokens at positions
        start, start+1, ... -> K, V [n, Hkv, dh]."""
        c = self.c
        ks, vs = [], []
        for i, t in enumerate(toks):
            _, _, k, v = self.sa_qkv(t, start + i)
            ks.append(k)
            vs.append(v)
        shape = (0, c["sa_hkv"], c["head_dim"])
        return (np.stack(ks) if ks else np.zeros(shape, F64),
                np.stack(vs) if vs else np.zeros(shape, F64))

    # ---- one drafter forward for one row ----------------------------------
    def forward_row(self, tok, pos, saK, saV, caK, caV, B, tliKV=None):
        """SA -> CA -> (TLI decoder layers) -> LM head for a token at position pos whose visible
        self-attention keys/values (excluding itself) are saK, saV; tliKV[l] = (K, V) visible to the row in
        TLI layer l (the LLM's cache of that layer, then the row's drafted ancestors).
        Returns dict(x, o_hat, ids, logp, k, v, z, tli_kv); o_hat is the input of the LM head."""
        e, q, k, v = self.sa_qkv(tok, pos)
        K = np.concatenate([np.asarray(saK, F64), k[None]], axis=0)
        V = np.concatenate([np.asarray(saV, F64), v[None]], axis=0)
        x = self.sa_block(e, q, K, V)
        o_hat = self.ca_block(x, caK, caV)
        tli_kv = []
        for l in range(self.tli_layers()):
            o_hat, kl, vl = self.tli_layer(l, o_hat, pos, tliKV[l][0], tliKV[l][1])
            tli_kv.append((kl, vl))
        ids, logp, z = self.head(o_hat, B)
        return dict(x=x, o_hat=o_hat, ids=ids, logp=logp, k=k, v=v, z=z, tli_kv=tli_kv)


# --------------------------------------------------------------------------
# the dynamic draft tree (Section 2.2, last paragraph)
# --------------------------------------------------------------------------
class TreeState:
    """Node pool of one sequence. Scores are fp32 sums of fp32 log-probs."""

    def __init__(self, root_tok, B, D, m):
        self.B, self.D, self.m = B, D, m
        self.root_tok = int(root_tok)
        self.tok, self.parent, self.depth = [], [], []   # parent: pool index or -1 (root)
        self.score = []                                  # np.float32
        self.step = 0
        self.frontier = [-1]                             # pool indices; -1 = root

    def frontier_tokens(self):
        return [self.root_tok if f < 0 else self.tok[f] for f in self.frontier]

    def path_to(self, node):
        """Pool indices from the depth-1 ancestor down to node (root excluded)."""
        path = []
        while node >= 0:
            path.append(node)
            node = self.parent[node]
        return path[::-1]


def tree_expand(ts: TreeState, ids, logp):
    """Append the children of the current frontier and choose the next one.

    ids, logp: [len(frontier), B], each row sorted as lm_head_topk sorts. A
    child's score is its parent's score plus its log-probability (fp32 add).
    Children are appended in (frontier row, rank) order; the next frontier is
    the top B of the new children by (score desc, pool index asc)."""
    B = ts.B
    logp = np.asarray(logp, np.float32)
    first = len(ts.tok)
    for r, f in enumerate(ts.frontier):
        base = np.float32(0.0) if f < 0 else ts.score[f]
        for j in range(B):
            ts.tok.append(int(ids[r][j]))
            ts.parent.append(f)
            ts.depth.append(ts.step + 1)
            ts.score.append(np.float32(base + logp[r][j]))
    new = list(range(first, len(ts.tok)))
    new.sort(key=lambda i: (-float(ts.score[i]), i))
    ts.frontier = new[:B]
    ts.step += 1


def tree_finalize(ts: TreeState):
    """Keep the min(m, pool) best nodes by (score desc, pool index asc), list
    them by pool index, put the root in slot 0 and rewrite parents as slots.
    Returns tok, parent, depth (int64 [n]) and score (float32 [n])."""
    n_pool = len(ts.tok)
    order = sorted(range(n_pool), key=lambda i: (-float(ts.score[i]), i))
    kept = sorted(order[:min(ts.m, n_pool)])
    slot = {-1: 0}
    for s, i in enumerate(kept):
        slot[i] = s + 1
    tok = [ts.root_tok] + [ts.tok[i] for i in kept]
    parent = [-1] + [slot[ts.parent[i]] for i in kept]
    depth = [0] + [ts.depth[i] for i in kept]
    score = [np.float32(0.0)] + [ts.score[i] for i in kept]
    return (np.array(tok, np.int64), np.array(parent, np.int64),
            np.array(depth, np.int64), np.array(score, np.float32))


def verify_greedy(tok, parent, target_logits):
    """Greedy (exact-match) verification of a kept draft tree (Section 2.2, step 2 with Tree Attention;
    Algorithm 1, the "identify K' verified tokens" step).

    tok, parent [n]: the kept tree, slot 0 = the root (last verified token), parent[0] = -1, parent[i] < i; an
    entry parent[i] < 0 at i > 0 marks an unused slot. target_logits [n, V]: the LLM's logits at every slot,
    row i scoring the token that follows slot i's token on its root path (one LLM pass with the tree mask).
    The LLM's choice at a slot is the arg-max (ties: smallest id). Starting at the root, the child carrying
    the chosen token is accepted and the walk continues from it; at the first slot with no such child
    everything else is discarded. Returns (slots, next_tok, choice): the accepted slots (root first, so
    K' = len(slots) - 1), the LLM's choice at the last accepted slot (the next cycle's root) and every
    slot's choice."""
    tok = [int(t) for t in tok]
    parent = [int(q) for q in parent]
    z = np.asarray(target_logits, F64)
    n = len(tok)
    choice = [int(np.lexsort((np.arange(z.shape[1]), -z[i]))[0]) for i in range(n)]
    slots = [0]
    cur = 0
    while True:
        nxt = [c for c in range(1, n) if parent[c] == cur and tok[c] == choice[cur]]
        if not nxt:
            break
        cur = nxt[0]
        slots.append(cur)
    return slots, choice[cur], choice


def tree_mask(parent):
    """mask[i][j] = 1 iff j == i or j is an ancestor of i. parent[0] = -1."""
    n = len(parent)
    mask = np.zeros((n, n), np.uint8)
    for i in range(n):
        j = i
        while j >= 0:
            mask[i, j] = 1
            j = int(parent[j])
    return mask


def draft_tree(dr: Drafter, root_tok, saK, saV, caK, caV, B, D, m, forced=None, tliK=None, tliV=None):
    """Grow one sequence's draft tree with D drafter forwards.

    saK, saV [ctx, Hkv, dh]: self-attention prefix cache (positions 0..ctx-1);
    the root sits at position ctx, a node of depth d at ctx + d, and sees the
    prefix, its ancestors (root included) and itself.
    forced: optional list of per-step (ids, logp) to expand with instead of
    the oracle's own top-B (used to follow another implementation's choices).
    tliK, tliV: per TLI layer, the LLM's cache of that layer over the same positions 0..ctx-1, [ctx, Hkv, dh];
    a node's keys / values in those layers are kept for the cycle and seen by its descendants (Section 3.2).
    Returns (TreeState, steps) with steps[s] = list of forward_row dicts."""
    ctx = saK.shape[0]
    ts = TreeState(root_tok, B, D, m)
    node_kv = {}      # pool index (or -1) -> (k, v) of nodes that were forwarded
    steps = []
    for s in range(D):
        rows = []
        for f in ts.frontier:
            # the root sees only the prefix; a node sees the root and its proper ancestors
            anc = [] if f < 0 else [-1] + ts.path_to(f)[:-1]
            Ks = [saK] + [node_kv[a][0][None] for a in anc]
            Vs = [saV] + [node_kv[a][1][None] for a in anc]
            tli = [(np.concatenate([tliK[l]] + [node_kv[a][2][l][0][None] for a in anc], 0),
                    np.concatenate([tliV[l]] + [node_kv[a][2][l][1][None] for a in anc], 0))
                   for l in range(dr.tli_layers())]
            tok = ts.root_tok if f < 0 else ts.tok[f]
            out = dr.forward_row(tok, ctx + s, np.concatenate(Ks, 0), np.concatenate(Vs, 0), caK, caV, B, tli)
            rows.append(out)
        for f, out in zip(ts.frontier, rows):
            node_kv[f] = (out["k"], out["v"], out["tli_kv"])
        steps.append(rows)
        if forced is not None:
            ids, logp = forced[s]
        else:
            ids = [r["ids"] for r in rows]
            logp = [r["logp"] for r in rows]
        tree_expand(ts, ids, logp)
    return ts, steps


# --------------------------------------------------------------------------
# independent loop-based paths used to pin the tree code by brute force
# --------------------------------------------------------------------------
def sequential_decode(dr: Drafter, prefix_toks, path_toks, caK, caV, B, tliK=None, tliV=None):
    """Plain causal decoding, token by token (Algorithm 1, the inner drafting loop with the
    tokens given): the self-attention cache grows by one entry per token and
    every token sees all earlier ones. Returns the forward_row dict of each
    token of path_toks."""
    c = dr.c
    K = np.zeros((0, c["sa_hkv"], c["head_dim"]), F64)
    V = np.zeros((0, c["sa_hkv"], c["head_dim"]), F64)
    pos = 0
    for t in prefix_toks:
        _, _, k, v = dr.sa_qkv(t, pos)
        K = np.concatenate([K, k[None]], 0)
        V = np.concatenate([V, v[None]], 0)
        pos += 1
    outs = []
    tli = [(np.asarray(tliK[l], F64), np.asarray(tliV[l], F64)) for l in range(dr.tli_layers())]
    for t in path_toks:
        out = dr.forward_row(t, pos, K, V, caK, caV, B, tli)
        K = np.concatenate([K, out["k"][None]], 0)
        V = np.concatenate([V, out["v"][None]], 0)
        tli = [(np.concatenate([tli[l][0], out["tli_kv"][l][0][None]], 0),
                np.concatenate([tli[l][1], out["tli_kv"][l][1][None]], 0)) for l in range(dr.tli_layers())]
        outs.append(out)
        pos += 1
    return outs


def drafter_prefill(dr: Drafter, toks, saK, saV, caK, caV, ca_limit=None):
    """The drafter over a whole token sequence in one pass (Section 3.1.2: the causal SA mask and the CA layer
    with its K-step-bounded mask, the pass the drafter is trained with): token i sits at position
    len(saK) + i, sees the prefix and tokens 0..i in self-attention, and the first ca_limit[i] cached LLM
    positions in cross-attention (None: all of them, the generation-time setting). TLI is not applied.
    Returns (o_hat [n, E], K, V) with K, V the self-attention cache extended by the n tokens."""
    c = dr.c
    K = np.asarray(saK, F64).reshape(-1, c["sa_hkv"], c["head_dim"])
    V = np.asarray(saV, F64).reshape(-1, c["sa_hkv"], c["head_dim"])
    outs = []
    for i, t in enumerate(toks):
        lim = len(caK) if ca_limit is None else int(ca_limit[i])
        e, q, k, v = dr.sa_qkv(int(t), K.shape[0])
        K = np.concatenate([K, k[None]], 0)
        V = np.concatenate([V, v[None]], 0)
        x = dr.sa_block(e, q, K, V)
        outs.append(dr.ca_block(x, caK[:lim], caV[:lim]))
    return (np.stack(outs) if outs else np.zeros((0, c["d_model"]), F64)), K, V


def greedy_chain(dr: Drafter, prefix_toks, root_tok, caK, caV, K_draft, tliK=None, tliV=None):
    """Chain drafting (Algorithm 1, inner loop) with greedy choice: K_draft
    tokens, each the most probable continuation. Returns (tokens, logps)."""
    toks, lps = [int(root_tok)], []
    for _ in range(K_draft):
        out = sequential_decode(dr, prefix_toks, toks, caK, caV, 1, tliK, tliV)[-1]
        toks.append(int(out["ids"][0]))
        lps.append(float(out["logp"][0]))
    return toks[1:], lps


# --------------------------------------------------------------------------
# client-server message codec (Section 4.2 "Client-Server"; message-size table in the appendix)
# --------------------------------------------------------------------------
def pack_tree(tok, parent):
    """Client message (Section 4.2): a draft-tree node takes four bytes, three for the token id (little endian) and
    the fourth for where the node sits in the tree, so a tree of M nodes is a message of 4M bytes, the size the
    message-size table gives.
    Reading: the fourth byte is the parent's slot number (a tree is its parent list; slots are < 255); 255
    marks "no parent" (the root, or an unused slot, whose token bytes are ff ff ff).
    tok, parent [n] -> uint8 [n, 4]."""
    n = len(tok)
    out = np.zeros((n, 4), np.uint8)
    for i in range(n):
        t, q = int(tok[i]), int(parent[i])
        t = 0xFFFFFF if t < 0 else t & 0xFFFFFF
        out[i] = [t & 0xFF, (t >> 8) & 0xFF, (t >> 16) & 0xFF, 255 if q < 0 else q & 0xFF]
    return out


def unpack_tree(msg):
    """Inverse of pack_tree: uint8 [n, 4] -> tok, parent (int64 [n]); ff ff ff -> token -1, 255 -> parent -1."""
    msg = np.asarray(msg, np.uint8)
    tok = msg[:, 0].astype(np.int64) | (msg[:, 1].astype(np.int64) << 8) | (msg[:, 2].astype(np.int64) << 16)
    tok[tok == 0xFFFFFF] = -1
    parent = msg[:, 3].astype(np.int64)
    parent[parent == 255] = -1
    return tok, parent


def quantize_rows(x):
    """8-bit quantisation of activation rows (Section 4.2: the E and E_kv tensors are quantised to 8 bits).
    Reading (the paper gives no scheme): symmetric, one fp32 scale per row, scale = max|x| / 127,
    code = round-half-even(x * (127 / max|x|)) in [-127, 127] -- one fp32 reciprocal per row, one fp32 product
    per element; an all-zero row has scale 0 and codes 0. The decision is taken in fp32 (the precision both
    sides use). x [rows, width] -> (int8 codes, float32 scales)."""
    x = np.asarray(x, np.float32)
    amax = np.max(np.abs(x), axis=-1).astype(np.float32)
    scale = (amax / np.float32(127.0)).astype(np.float32)
    nz = amax > 0
    inv = np.where(nz, np.float32(127.0) / np.where(nz, amax, np.float32(1.0)), np.float32(0.0)).astype(np.float32)
    q = np.rint((x * inv[:, None]).astype(np.float32))
    q = np.clip(q, -127, 127)
    return q.astype(np.int8), scale


def dequantize_rows(codes, scales):
    """x ~ code * scale, one fp32 product per element."""
    return (np.asarray(codes, np.float32) * np.asarray(scales, np.float32)[:, None]).astype(np.float32)
