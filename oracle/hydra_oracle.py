"""CPU oracle of one Hydra speculative-decode step.  TEST INFRASTRUCTURE, not a product path.

Plain, slow, step-by-step restatement of the method in torch CPU ops, used only by the tests, the
smoke check and the CPU-baseline leg of the benchmark.  It shares no code with the CUDA library and
imports nothing from it.  Arithmetic runs in `dtype` (float64 by default; float32 for the large
shapes, where the weights are bfloat16-rounded values widened on use).

What it follows (Hydra: Sequentially-Dependent Draft Heads for Medusa Decoding):
  * Background, "Speculative decoding": draft, verify in one base forward, accept a prefix.
  * Background, "Tree decoding": static candidate tree, children = top-m tokens in descending
    probability, one packed forward where a token attends only to its ancestors.
  * Section "Hydra Heads", second displayed equation: head i is a function of the last hidden
    state, x_t and the i-1 tokens speculated before it, concatenated on the feature dimension.
  * Section "Hydra++": MLP depth 4 and one extra decoder layer queried once per step.
  * Background, "Lightweight heads as a draft model" / "Medusa decoding": the baseline whose head i is a
    function of the hidden state alone (head.medusa).
  * Background, verification criteria: greedy acceptance (a candidate is kept when it equals the
    base model's most likely token).
  * Section "Typical acceptance sampling", paragraph "Typical acceptance criterion": a candidate is
    kept when its probability under the temperature-tau base distribution at its parent exceeds
    min(epsilon, alpha * exp(-entropy of that distribution)).

Pinned by tests/test_oracle_*.py: a whole-model comparison against the `transformers` Llama
implementation, chain-tree == token-by-token decoding, root-only tree == greedy decoding, output
invariance to the drafted tokens, brute-force acceptance, compaction == sequential decoding,
closed-form head cases, library sort for top-k, brute-force ancestor masks; the typical criterion by its
limits (tau -> 0 is the greedy criterion, epsilon -> 0 keeps every candidate, a uniform row has
entropy log V), a library entropy routine and brute force over the tree's paths.
Parity unpinned: the numeric values of logits for the random models (the paper prints none); they
are fixed only by the pins above on the operations that produce them.
"""
from typing import Dict, List, Optional, Sequence
import math
import torch


# ----------------------------------------------------------------------------- tree tables
class TreeTables:
    """Static tables of a candidate tree (Background, "Tree decoding").

    parent[0] = -1 is the root (the committed token x_t not yet run through the base model);
    every other row is a candidate token.  Tables are built by walking parent[] upward.
    """

    def __init__(self, parent: Sequence[int], max_depth: Optional[int] = None):
        T = len(parent)
        if T < 1 or T > 64 or parent[0] != -1:
            raise ValueError("tree needs 1..64 rows and parent[0] == -1")
        self.parent = list(parent)
        self.T = T
        self.depth = [0] * T
        self.children: List[List[int]] = [[] for _ in range(T)]
        for i in range(1, T):
            p = parent[i]
            if not (0 <= p < i):
                raise ValueError("parent[i] must satisfy 0 <= parent[i] < i")
            self.depth[i] = self.depth[p] + 1
            self.children[p].append(i)
        self.rank_path = [()] * T
        for i in range(1, T):
            p = parent[i]
            self.rank_path[i] = self.rank_path[p] + (self.children[p].index(i),)
        keys = [(self.depth[i], self.rank_path[i]) for i in range(T)]
        if keys != sorted(keys):
            raise ValueError("rows must be ordered by (depth, rank path)")
        self.K = max(self.depth)
        if max_depth is not None and self.K > max_depth:
            raise ValueError("tree deeper than the number of heads")
        # path[i] = rows from the root down to i
        self.path = []
        for i in range(T):
            rows, j = [], i
            while j != -1:
                rows.append(j)
                j = parent[j]
            self.path.append(rows[::-1])
        # allowed[i][j]: row i may attend to tree row j  <=>  j is an ancestor of i or i itself
        self.allowed = torch.zeros(T, T, dtype=torch.bool)
        for i in range(T):
            for j in self.path[i]:
                self.allowed[i, j] = True
        self.anc_mask = [sum(1 << j for j in self.path[i]) for i in range(T)]
        # parents that have children, per level d = 1..K (the rows head d is queried at)
        self.level_parents = [[i for i in range(T) if self.depth[i] == d - 1 and self.children[i]]
                              for d in range(1, self.K + 1)]


# ----------------------------------------------------------------------------- sub-blocks
def rmsnorm(x: torch.Tensor, w: torch.Tensor, eps: float) -> torch.Tensor:
    """x * w / sqrt(mean(x^2) + eps), row-wise (Llama RMSNorm)."""
    return x * torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps) * w


def rope(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding, half-split pairing: (x_i, x_{i+hd/2}) rotated by pos * theta^(-2i/hd).

    x: [n, H, hd], pos: [n] integer positions.
    """
    hd = x.shape[-1]
    half = hd // 2
    inv = theta ** (-torch.arange(0, half, dtype=torch.float64) * 2.0 / hd)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]                   # [n, half]
    c, s = torch.cos(ang).to(x.dtype)[:, None, :], torch.sin(ang).to(x.dtype)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return torch.cat([a * c - b * s, b * c + a * s], dim=-1)


def silu(x: torch.Tensor) -> torch.Tensor:
    return x / (1.0 + torch.exp(-x))


def masked_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, mask: torch.Tensor) -> torch.Tensor:
    """softmax(q k^T / sqrt(hd) restricted to mask) v per head.  q: [n, H, hd]; k, v: [L, H, hd];
    mask: [n, L] bool (row i may attend to slot j).  Returns [n, H, hd]."""
    scores = torch.einsum("nhd,lhd->hnl", q, k) / math.sqrt(q.shape[-1])
    scores = scores.masked_fill(~mask[None], float("-inf"))
    return torch.einsum("hnl,lhd->nhd", torch.softmax(scores, dim=-1), v)


def topk_desc(logits: torch.Tensor, k: int) -> List[int]:
    """The k most likely tokens in descending order; equal logits ordered by ascending token id."""
    vals = logits.tolist()
    order = sorted(range(len(vals)), key=lambda t: (-vals[t], t))
    return order[:k]


def argmax_lowest(logits: torch.Tensor) -> torch.Tensor:
    """Row-wise argmax, lowest index among equal maxima.  logits: [n, V] -> [n] int64."""
    mx = logits.max(dim=-1, keepdim=True).values
    V = logits.shape[-1]
    idx = torch.arange(V).expand_as(logits)
    return torch.where(logits == mx, idx, torch.full_like(idx, V)).min(dim=-1).values


def typical_row(logits: torch.Tensor, tau: float, eps: float, alpha: float):
    """One parent's side of the typical acceptance criterion (Section "Typical acceptance sampling",
    displayed inequality): p = softmax(logits / tau), H = -sum p log p, threshold = min(eps, alpha * exp(-H)).
    Returns (p, threshold); a child token x is accepted when p[x] > threshold."""
    z = logits.double() / tau
    z = z - z.max()
    e = torch.exp(z)
    p = e / e.sum()
    logp = z - torch.log(e.sum())
    H = -(p * logp).sum()                      # p = 0 terms vanish: exp underflow gives 0 * finite
    return p, min(eps, alpha * math.exp(-float(H)))


def inverse_cdf(p: torch.Tensor, u: float) -> int:
    """The token drawn from p by the uniform number u in [0, 1): the first id whose cumulative probability
    (in token-id order) exceeds u."""
    c = torch.cumsum(p.double(), dim=0)
    idx = int((c > u * float(c[-1])).nonzero()[0])
    return idx


# ----------------------------------------------------------------------------- the oracle
class HydraOracle:
    """State and phases of Hydra decoding for a batch of independent sequences."""

    def __init__(self, model, head, parent: Sequence[int], weights: Dict[str, torch.Tensor],
                 max_seq: int, dtype=torch.float64, cache_weights=False):
        self.m, self.h = model, head
        self.tree = TreeTables(parent, max_depth=head.n_heads)
        self.w = weights
        self.dtype = dtype
        self.max_seq = max_seq
        self.B = 0
        self._wcache: Dict[str, torch.Tensor] = {}
        self._cache_weights = cache_weights
        self.hprime: List[torch.Tensor] = []

    def W(self, name: str) -> torch.Tensor:
        """Weight `name` widened to the arithmetic dtype (head, embedding and LM-head matrices, which
        are used many times per step, are kept widened when cache_weights is True, everything when it is "all";
        the rest is widened on use)."""
        if name in self._wcache:
            return self._wcache[name]
        t = self.w[name].to(device="cpu", dtype=self.dtype)
        if self._cache_weights == "all" or (self._cache_weights and (name[0] == "H" or name in ("embed", "lm_head"))):
            self._wcache[name] = t
        return t

    # -- one Llama decoder layer over n new rows of one sequence, appending to that layer's cache
    def _layer(self, pre: str, x, pos, allowed_new, kc, vc, cache_len):
        """x: [n, d] residual rows; pos: [n]; allowed_new: [n, n] bool among the new rows;
        kc, vc: [max_seq, H, hd] caches holding cache_len committed rows.  New rows are written at
        slots cache_len + i; row i attends to every committed slot and to allowed new rows."""
        m = self.m
        n, H, hd = x.shape[0], m.n_heads, m.head_dim
        xn = rmsnorm(x, self.W(pre + "attn_norm"), m.rms_eps)
        qkv = xn @ self.W(pre + "wqkv").T
        q, k, v = [t.reshape(n, H, hd) for t in qkv.split(m.d_model, dim=-1)]
        q, k = rope(q, pos, m.rope_theta), rope(k, pos, m.rope_theta)
        kc[cache_len:cache_len + n] = k
        vc[cache_len:cache_len + n] = v
        L = cache_len + n
        mask = torch.cat([torch.ones(n, cache_len, dtype=torch.bool), allowed_new], dim=1)   # [n, L]
        att = masked_attention(q, kc[:L], vc[:L], mask).reshape(n, m.d_model)
        x = x + att @ self.W(pre + "wo").T
        xn = rmsnorm(x, self.W(pre + "ffn_norm"), m.rms_eps)
        gu = xn @ self.W(pre + "w_gate_up").T
        g, u = gu.split(m.d_ffn, dim=-1)
        return x + (silu(g) * u) @ self.W(pre + "w_down").T

    def _base_rows(self, b, tok, pos, allowed_new):
        """Base-model forward of n new rows of sequence b on top of its cache (not committed)."""
        x = self.W("embed")[tok.long()]
        for l in range(self.m.n_layers):
            x = self._layer(f"L{l}.", x, pos, allowed_new, self.kc[l][b], self.vc[l][b], self.len[b])
        return rmsnorm(x, self.W("final_norm"), self.m.rms_eps)        # post-final-norm hidden rows

    # -- prefill: ordinary causal forward over the prompt
    def prefill(self, prompts: List[torch.Tensor]):
        m = self.m
        B = self.B = len(prompts)
        shape = (self.max_seq, m.n_heads, m.head_dim)
        self.kc = [[torch.zeros(shape, dtype=self.dtype) for _ in range(B)] for _ in range(m.n_layers)]
        self.vc = [[torch.zeros(shape, dtype=self.dtype) for _ in range(B)] for _ in range(m.n_layers)]
        self.pk = [torch.zeros(shape, dtype=self.dtype) for _ in range(B)]       # prefix-layer cache
        self.pv = [torch.zeros(shape, dtype=self.dtype) for _ in range(B)]
        self.len = [0] * B
        self.root_tok = [0] * B
        self.h_new: List[torch.Tensor] = [None] * B
        for b, p in enumerate(prompts):
            n = p.numel()
            causal = torch.tril(torch.ones(n, n, dtype=torch.bool))
            h = self._base_rows(b, p, torch.arange(n), causal)
            self.len[b] = n
            self.h_new[b] = h                                           # all prompt rows feed the prefix layer
            self.root_tok[b] = int(argmax_lowest(h[-1:] @ self.W("lm_head").T)[0])

    # -- draft: prefix layer once, then the heads level by level
    def _head_input_hidden(self, b):
        """h': the hidden state the heads consume.  Hydra++: output of the extra decoder layer at the
        last committed position, run over the rows committed since its last call (Section Hydra++,
        "Prefix Attention"); otherwise the base model's last hidden state."""
        hn = self.h_new[b]
        if not self.h.prefix_attn:
            return hn[-1]
        n = hn.shape[0]
        pos = torch.arange(self.len[b] - n, self.len[b])
        causal = torch.tril(torch.ones(n, n, dtype=torch.bool))
        # the prefix-layer cache holds every committed row older than the rows in h_new
        return self._layer("P.", hn, pos, causal, self.pk[b], self.pv[b], self.len[b] - n)[-1]

    def head_logits(self, i: int, hprime: torch.Tensor, path_tok: Sequence[int]) -> torch.Tensor:
        """Hydra head i (1-based) at one parent: MLP over [h' ; E[x_t] ; E[x^_{t+1}] ...] then the
        shared LM head.  path_tok = tokens on the path root..parent (i of them).  A sequentially
        independent (Medusa) head sees h' alone, so all parents of a level get the same distribution."""
        assert len(path_tok) == i
        E = self.W("embed")
        z = hprime if getattr(self.h, "medusa", False) else torch.cat([hprime] + [E[t] for t in path_tok])
        y = hprime + silu(self.W(f"H{i}.w1") @ z + self.W(f"H{i}.b1"))
        for l in range(self.h.n_mlp_layers - 1):
            y = y + silu(self.W(f"H{i}.wr")[l] @ y + self.W(f"H{i}.br")[l])
        return self.W("lm_head") @ y

    def draft(self, return_logits: bool = False):
        """Populate the candidate tree: children of a parent = its head's top-c tokens, descending."""
        t = self.tree
        tok = torch.zeros(self.B, t.T, dtype=torch.int64)
        all_logits = [dict() for _ in range(self.B)]
        self.hprime = []
        for b in range(self.B):
            hp = self._head_input_hidden(b)
            self.hprime.append(hp)
            tok[b, 0] = self.root_tok[b]
            for d in range(1, t.K + 1):
                for p in t.level_parents[d - 1]:
                    lg = self.head_logits(d, hp, [int(tok[b, j]) for j in t.path[p]])
                    all_logits[b][p] = lg
                    for c, tk in zip(t.children[p], topk_desc(lg, len(t.children[p]))):
                        tok[b, c] = tk
        return (tok, all_logits) if return_logits else tok

    # -- verify: one base forward over all tree rows with the ancestor mask
    def verify(self, tree_tok: torch.Tensor):
        t = self.tree
        self.h_tree, logits, amax = [], [], []
        for b in range(self.B):
            pos = self.len[b] + torch.tensor(t.depth)
            h = self._base_rows(b, tree_tok[b], pos, t.allowed)
            lg = h @ self.W("lm_head").T
            self.h_tree.append(h)
            logits.append(lg)
            amax.append(argmax_lowest(lg))
        return torch.stack(amax), torch.stack(logits)

    # -- acceptance + cache compaction
    def _commit(self, b: int, best: int, new_root: int, tree_tok: torch.Tensor):
        """Append the accepted path root..best of sequence b to its state: the accepted rows' K,V move next to the
        committed prefix (everything else in the tree is dropped), their hidden rows feed the next draft."""
        t = self.tree
        path = t.path[best]
        n = len(path) - 1
        L = self.len[b]
        for l in range(self.m.n_layers):
            for cache in (self.kc[l][b], self.vc[l][b]):
                moved = cache[L + torch.tensor(path)].clone()        # out of place
                cache[L:L + n + 1] = moved
        self.h_new[b] = self.h_tree[b][path].clone()
        self.len[b] = L + n + 1
        self.root_tok[b] = new_root
        K = self.h.n_heads
        out = [int(tree_tok[b, j]) for j in path[1:]] + [new_root]
        return n, path + [-1] * (K + 1 - len(path)), out + [-1] * (K + 1 - len(out))

    def _deepest(self, accepted: List[bool]) -> int:
        """The deepest accepted row, the lowest row index among equals."""
        t = self.tree
        best = 0
        for i in range(t.T):
            if accepted[i] and t.depth[i] > t.depth[best]:
                best = i
        return best

    def accept_compact(self, tree_tok: torch.Tensor, amax: torch.Tensor):
        """Greedy criterion: a candidate is accepted when it equals the base argmax at its parent and its parent is
        accepted; the deepest accepted row wins (lowest row index among equals)."""
        t = self.tree
        n_acc, paths, outs = [], [], []
        for b in range(self.B):
            accepted = [True] + [False] * (t.T - 1)
            for i in range(1, t.T):                       # parents precede children
                p = t.parent[i]
                accepted[i] = accepted[p] and int(tree_tok[b, i]) == int(amax[b, p])
            best = self._deepest(accepted)
            n, path, out = self._commit(b, best, int(amax[b, best]), tree_tok)
            n_acc.append(n); paths.append(path); outs.append(out)
        return torch.tensor(n_acc), torch.tensor(paths), torch.tensor(outs)

    def typical_pass(self, tree_tok: torch.Tensor, logits: torch.Tensor, tau: float, eps: float, alpha: float):
        """[B][T] bool: candidate i passes the typical criterion at its parent (row 0 is True).  Also returns the
        margin log p - log threshold of every candidate (how far the decision is from flipping)."""
        t = self.tree
        ok = torch.ones(self.B, t.T, dtype=torch.bool)
        margin = torch.full((self.B, t.T), float("inf"), dtype=torch.float64)
        for b in range(self.B):
            rows = {}
            for i in range(1, t.T):
                par = t.parent[i]
                if par not in rows:
                    rows[par] = typical_row(logits[b, par], tau, eps, alpha)
                p, thr = rows[par]
                px = float(p[int(tree_tok[b, i])])
                ok[b, i] = px > thr
                margin[b, i] = (math.log(px) if px > 0 else -1e30) - math.log(thr)
        return ok, margin

    def typical_accept_compact(self, tree_tok: torch.Tensor, logits: torch.Tensor, tau: float, eps: float, alpha: float,
                               u: Optional[Sequence[float]] = None):
        """Typical acceptance (Section "Typical acceptance sampling"): a candidate is accepted when it passes the
        criterion at its parent and its parent is accepted; the deepest accepted row wins (lowest row index among
        equals).  The token after the accepted path comes from the temperature-tau base distribution at the best
        row: drawn by inverse CDF with the uniform number u[b], or its most likely token when u is None."""
        t = self.tree
        ok, _ = self.typical_pass(tree_tok, logits, tau, eps, alpha)
        n_acc, paths, outs = [], [], []
        for b in range(self.B):
            accepted = [True] + [False] * (t.T - 1)
            for i in range(1, t.T):
                accepted[i] = accepted[t.parent[i]] and bool(ok[b, i])
            best = self._deepest(accepted)
            if u is None:
                new_root = int(argmax_lowest(logits[b, best:best + 1])[0])
            else:
                new_root = inverse_cdf(typical_row(logits[b, best], tau, eps, alpha)[0], float(u[b]))
            n, path, out = self._commit(b, best, new_root, tree_tok)
            n_acc.append(n); paths.append(path); outs.append(out)
        return torch.tensor(n_acc), torch.tensor(paths), torch.tensor(outs)

    def step(self, plant: Optional[torch.Tensor] = None):
        tok = self.draft()
        if plant is not None:
            tok = torch.where(plant >= 0, plant, tok)
        amax, _ = self.verify(tok)
        return self.accept_compact(tok, amax)

    # -- plain greedy decoding, one token per base forward (the autoregressive baseline)
    def greedy_continuation(self, b: int, n_tokens: int) -> List[int]:
        """Tokens the base model emits greedily after the committed prefix of sequence b (the first is
        root_tok).  Runs on copies of the caches; the oracle's state is left untouched."""
        saved = ([c[b].clone() for c in self.kc], [c[b].clone() for c in self.vc], self.len[b])
        out, tok = [self.root_tok[b]], self.root_tok[b]
        one = torch.ones(1, 1, dtype=torch.bool)
        for _ in range(n_tokens - 1):
            h = self._base_rows(b, torch.tensor([tok]), torch.tensor([self.len[b]]), one)
            self.len[b] += 1
            tok = int(argmax_lowest(h @ self.W("lm_head").T)[0])
            out.append(tok)
        for l in range(self.m.n_layers):
            self.kc[l][b], self.vc[l][b] = saved[0][l], saved[1][l]
        self.len[b] = saved[2]
        return out
