"""A toy attention-only language model used to check losslessness end to end.

The parts of a decoding round that lie outside the library (embeddings, Q/K/V/O
projections, lm-head, building the draft tree) are evaluated here in numpy fp64 with
random weights.  The four library operations are supplied by an ``ops`` object, so the
same loop runs against the CPU oracle and against the CUDA library.  The claim under
test is the paper's (Section "Setup"): with greedy sampling, draft-and-verify rounds
emit exactly the tokens of plain auto-regressive decoding, and (our addition) the
compacted KV cache equals the auto-regressive cache.
"""
import numpy as np


class ToyLM:
    def __init__(self, seed=0, V=50, d=32, layers=2, Hq=4, Hkv=2, D=8, max_pos=256, k_steps=2,
                 transfer_after=1):
        rng = np.random.default_rng(seed)
        self.V, self.d, self.layers, self.Hq, self.Hkv, self.D = V, d, layers, Hq, Hkv, D
        self.E = rng.standard_normal((V, d))
        self.Pos = 0.5 * rng.standard_normal((max_pos, d))
        s = 1.0 / np.sqrt(d)
        self.Wq = rng.standard_normal((layers, d, Hq * D)) * s * 2.0
        self.Wk = rng.standard_normal((layers, d, Hkv * D)) * s * 2.0
        self.Wv = rng.standard_normal((layers, d, Hkv * D)) * s
        self.Wo = rng.standard_normal((layers, Hq * D, d)) * s
        self.Wt = rng.standard_normal((k_steps, d, d)).astype(np.float32) * np.float32(s)
        self.k_steps = k_steps
        self.transfer_after = transfer_after      # pseudo rows exist from this layer index on

    # ---- plain auto-regressive greedy decoding, independent of the library and the oracle ----
    def ar_decode(self, prompt, n_new):
        cache_k = [np.zeros((self.Hkv, 0, self.D), np.float32) for _ in range(self.layers)]
        cache_v = [np.zeros((self.Hkv, 0, self.D), np.float32) for _ in range(self.layers)]
        g = self.Hq // self.Hkv
        tokens = list(prompt)
        out = []
        pos = 0
        nxt = None
        feed = list(prompt)
        while len(out) < n_new:
            for t in feed:
                x = self.E[t] + self.Pos[pos]
                for l in range(self.layers):
                    q = (x @ self.Wq[l]).astype(np.float32).reshape(self.Hq, self.D)
                    kk = (x @ self.Wk[l]).astype(np.float32).reshape(self.Hkv, 1, self.D)
                    vv = (x @ self.Wv[l]).astype(np.float32).reshape(self.Hkv, 1, self.D)
                    cache_k[l] = np.concatenate([cache_k[l], kk], axis=1)
                    cache_v[l] = np.concatenate([cache_v[l], vv], axis=1)
                    heads = []
                    for h in range(self.Hq):
                        s = cache_k[l][h // g].astype(np.float64) @ q[h].astype(np.float64)
                        s = s / np.sqrt(self.D)
                        w = np.exp(s - s.max())
                        w /= w.sum()
                        heads.append(w @ cache_v[l][h // g].astype(np.float64))
                    x = x + np.concatenate(heads) @ self.Wo[l]
                pos += 1
                nxt = int(np.argmax(x @ self.E.T))
            out.append(nxt)
            tokens.append(nxt)
            feed = [nxt]
        return out, cache_k, cache_v

    # ---- one forward over flattened tree rows using the library operations ----
    def tree_forward(self, ops, tokens_rows, positions, parent, src, k_cache, v_cache, kv_len):
        """tokens_rows/positions: per-sequence lists for the T tree rows; parent [B, T+P];
        caches [layers, B, Hkv, cap, D] float32 are written at rows kv_len[b] + r."""
        B = len(tokens_rows)
        T = len(tokens_rows[0])
        P = self.k_steps
        x = np.stack([self.E[np.array(tokens_rows[b])] + self.Pos[np.array(positions[b])]
                      for b in range(B)])                                   # [B, T, d]
        for l in range(self.layers):
            if l == self.transfer_after:
                h_src = np.stack([x[b, src[b]] for b in range(B)]).astype(np.float32)
                pseudo = np.asarray(ops.transfer(h_src, self.Wt), dtype=np.float64)  # [B, P, d]
                x = np.concatenate([x, pseudo], axis=1)
            rows = x.shape[1]
            q = (x @ self.Wq[l]).astype(np.float32).reshape(B, rows, self.Hq, self.D)
            kk = (x @ self.Wk[l]).astype(np.float32).reshape(B, rows, self.Hkv, self.D)
            vv = (x @ self.Wv[l]).astype(np.float32).reshape(B, rows, self.Hkv, self.D)
            for b in range(B):
                k_cache[l, b, :, kv_len[b]:kv_len[b] + rows] = kk[b].transpose(1, 0, 2)
                v_cache[l, b, :, kv_len[b]:kv_len[b] + rows] = vv[b].transpose(1, 0, 2)
            par = np.ascontiguousarray(parent[:, :rows])
            att = np.asarray(ops.attention(q, k_cache[l], v_cache[l], kv_len, par), dtype=np.float64)
            x = x + att.reshape(B, rows, self.Hq * self.D) @ self.Wo[l]
        assert x.shape[1] == T + P
        return x @ self.E.T                                                  # logits [B, T+P, V]


def make_draft_tree(rng, truth, depth, branch, p_true, V, with_root):
    """Candidate tree around the true continuation: at each level every frontier node gets
    ``branch`` children with distinct tokens; with probability ``p_true`` one of the children
    of the node on the true path carries the true next token."""
    parent, tokens, level = [], [], []
    on_truth = {}
    if with_root:
        parent.append(-1)
        tokens.append(truth[0])
        level = [0]
        on_truth[0] = 1                      # number of true tokens consumed along this node's path
        start = 1
    else:
        level = [-1]
        on_truth[-1] = 0
        start = 0
    for _ in range(depth):
        nxt = []
        for node in level:
            toks = list(rng.choice(V, size=branch, replace=False))
            if node in on_truth and on_truth[node] < len(truth):
                want = truth[on_truth[node]]
                if rng.random() < p_true:
                    if want in toks:
                        toks.remove(want)
                    else:
                        toks.pop()
                    toks.insert(int(rng.integers(branch)), want)
                else:
                    toks = [t if t != want else (t + 1) % V for t in toks]
                    if len(set(toks)) < branch:
                        toks = [(want + 1 + i) % V for i in range(branch)]
            for t in toks:
                c = len(parent)
                parent.append(node)
                tokens.append(int(t))
                nxt.append(c)
                if node in on_truth and on_truth[node] < len(truth) and t == truth[on_truth[node]]:
                    on_truth[c] = on_truth[node] + 1
        level = nxt
    return np.array(parent, np.int32), np.array(tokens, np.int32)


def single_token_parent(P):
    """One real row followed by its chain of P pseudo rows."""
    return np.array([[-1] + list(range(P))], np.int32)


def run_lossless_loop(ops, with_root, seed=0, n_new=24, atol_cache=1e-5, D=8):
    """Tree-verify rounds against plain greedy decoding for two sequences with different
    prompt lengths.  Returns the number of rounds used (fewer than n_new means drafts were
    accepted)."""
    lm = ToyLM(seed, D=D)
    rng = np.random.default_rng(seed + 100)
    prompts = [list(rng.integers(0, lm.V, 5)), list(rng.integers(0, lm.V, 9))]
    B = len(prompts)
    truth, ar_k, ar_v = [], [], []
    for p in prompts:
        t, ck, cv = lm.ar_decode(p, n_new + 8)
        truth.append(t)
        ar_k.append(ck)
        ar_v.append(cv)
    depth, branch = 3, 2
    T = (1 if with_root else 0) + sum(branch ** (i + 1) for i in range(depth))
    P = lm.k_steps
    N = T + P
    cap = max(len(p) for p in prompts) + n_new + 16 + N
    k_cache = np.zeros((lm.layers, B, lm.Hkv, cap, lm.D), np.float32)
    v_cache = np.zeros_like(k_cache)
    # prefill = a chain "tree" holding the prompt minus its last token, accepted wholesale
    kv_len = np.zeros(B, np.int32)
    generated = [[] for _ in range(B)]
    pending = [None] * B                        # the known-correct next token per sequence
    for b in range(B):
        for i, t in enumerate(prompts[b]):
            chain_parent = single_token_parent(P)
            logits = lm.tree_forward(ops, [[t]], [[i]], chain_parent, [0],
                                     k_cache[:, b:b + 1], v_cache[:, b:b + 1], kv_len[b:b + 1])
            kv_len[b] += 1
            pending[b] = int(np.argmax(logits[0, 0]))
        assert pending[b] == truth[b][0]
    rounds = 0
    while min(len(g) for g in generated) < n_new:
        rounds += 1
        parents, toks, positions = [], [], []
        for b in range(B):
            done = len(generated[b])
            future = truth[b][done:done + depth + 1]
            par, tk = make_draft_tree(rng, future, depth, branch, 0.7, lm.V, with_root)
            dep = np.zeros(len(par), np.int32)
            for c, p_ in enumerate(par):
                dep[c] = 0 if p_ < 0 else dep[p_] + 1
            parents.append(np.concatenate([par, [0] + [T + i for i in range(P - 1)]]).astype(np.int32))
            toks.append(tk)
            positions.append(list(int(kv_len[b]) + dep))
        parent = np.stack(parents)
        tokens = np.stack(toks)
        logits = lm.tree_forward(ops, [list(t) for t in tokens], positions, parent, [0] * B,
                                 k_cache, v_cache, kv_len)
        root_pred = None if with_root else np.array(pending, np.int32)
        pred, alen, apath, nxt, status = ops.verify(logits.astype(np.float32), tokens, parent,
                                                    root_pred, 8)
        assert (np.asarray(status) == 0).all()
        k_cache, v_cache, new_len = ops.compact(k_cache, v_cache, N, kv_len, alen, apath)
        for b in range(B):
            accepted = [int(tokens[b, c]) for c in apath[b, :alen[b]]]
            if not with_root and alen[b] == 0:
                # nothing drafted was right: feed the known next token alone next round
                one = single_token_parent(P)
                lg = lm.tree_forward(ops, [[pending[b]]], [[int(kv_len[b])]], one, [0],
                                     k_cache[:, b:b + 1], v_cache[:, b:b + 1], kv_len[b:b + 1])
                generated[b].append(pending[b])
                pending[b] = int(np.argmax(lg[0, 0]))
                kv_len[b] += 1
                continue
            generated[b].extend(accepted)
            pending[b] = int(nxt[b])
            kv_len[b] = new_len[b]
    for b in range(B):
        n = min(len(generated[b]), len(truth[b]))
        assert generated[b][:n] == truth[b][:n], "tree-verify decoding diverged from greedy decoding"
        rows = min(int(kv_len[b]), ar_k[b][0].shape[1])
        for l in range(lm.layers):
            assert np.abs(k_cache[l, b, :, :rows] - ar_k[b][l][:, :rows]).max() < atol_cache
            assert np.abs(v_cache[l, b, :, :rows] - ar_v[b][l][:, :rows]).max() < atol_cache
    return rounds
