"""Independent evaluator used to pin the oracle: library fp64 modules, whole prefix re-run.

Nothing here is shared with the oracle or with the CUDA path.  The prediction
network is ``torch.nn.LSTM`` run from a zero state over the full token history
(start-of-sequence blank + prefix) every time it is asked for -- the opposite of
the oracle's incremental, stateful update -- and the linear layers are
``torch.nn.functional.linear`` in fp64.
"""
import numpy as np
import torch


class NaiveModel:
    def __init__(self, w):
        self.w = w
        self.E, self.P, self.L = int(w["E"]), int(w["P"]), int(w["L"])
        self.blank = int(w["blank_id"])
        self.act = int(w["act"])
        self.emb = torch.tensor(np.asarray(w["emb"]), dtype=torch.float64)
        self.lstm = torch.nn.LSTM(self.E, self.P, num_layers=self.L).double()
        with torch.no_grad():
            for l in range(self.L):
                getattr(self.lstm, f"weight_ih_l{l}").copy_(torch.tensor(np.asarray(w["w_ih"][l]), dtype=torch.float64))
                getattr(self.lstm, f"weight_hh_l{l}").copy_(torch.tensor(np.asarray(w["w_hh"][l]), dtype=torch.float64))
                getattr(self.lstm, f"bias_ih_l{l}").copy_(torch.tensor(np.asarray(w["b_ih"][l]), dtype=torch.float64))
                getattr(self.lstm, f"bias_hh_l{l}").copy_(torch.tensor(np.asarray(w["b_hh"][l]), dtype=torch.float64))
        t = lambda k: torch.tensor(np.asarray(w[k]), dtype=torch.float64)
        self.w_enc, self.b_enc = t("w_enc"), t("b_enc")
        self.w_pred, self.b_pred = t("w_pred"), t("b_pred")
        self.w_out, self.b_out = t("w_out"), t("b_out")

    @torch.no_grad()
    def decoder(self, prefix):
        toks = torch.tensor([self.blank] + [int(p) for p in prefix], dtype=torch.long)
        out, (h, c) = self.lstm(self.emb[toks].unsqueeze(1))
        return out[-1, 0], h[:, 0], c[:, 0]

    @torch.no_grad()
    def logits(self, enc_t, prefix):
        h_top, _, _ = self.decoder(prefix)
        g = torch.nn.functional.linear(h_top, self.w_pred, self.b_pred)
        e = torch.nn.functional.linear(torch.tensor(np.asarray(enc_t), dtype=torch.float64), self.w_enc, self.b_enc)
        s = e + g
        z = torch.relu(s) if self.act == 0 else torch.tanh(s)
        return torch.nn.functional.linear(z, self.w_out, self.b_out).numpy()


def random_weights(rng, D, E, P, L, H, V, blank_id=None, act=0, blank_bias=0.0, bias_scale=0.0, emb_zero_blank=True):
    """Small random model in the same dict format as the input generator's."""
    blank_id = V if blank_id is None else blank_id
    n = lambda *s: rng.standard_normal(s).astype(np.float32)
    emb = n(V + 1, E)
    if emb_zero_blank:
        emb[blank_id] = 0
    w = dict(D=D, E=E, P=P, L=L, H=H, V=V, blank_id=blank_id, act=act, dtype="f32", emb=emb,
             w_ih=[n(4 * P, E if l == 0 else P) / np.sqrt(E if l == 0 else P) for l in range(L)],
             w_hh=[n(4 * P, P) / np.sqrt(P) for l in range(L)],
             b_ih=[bias_scale * n(4 * P) for l in range(L)], b_hh=[bias_scale * n(4 * P) for l in range(L)],
             w_enc=n(H, D) / np.sqrt(D), b_enc=bias_scale * n(H),
             w_pred=n(H, P) / np.sqrt(P), b_pred=bias_scale * n(H),
             w_out=n(V + 1, H) / np.sqrt(H), b_out=bias_scale * n(V + 1))
    w["b_out"][blank_id] += np.float32(blank_bias)
    for k, v in list(w.items()):
        if isinstance(v, np.ndarray):
            w[k] = v.astype(np.float32)
        elif isinstance(v, list):
            w[k] = [a.astype(np.float32) for a in v]
    return w


# ---------------------------------------------------------------------------
# A model whose logits are set by hand, with EXACT ties, to pin the argmax tie rule (lowest index wins).
# ---------------------------------------------------------------------------
TIE_TYPES = 9   # frame types of tie_model


def tie_model(V=299, blank_id=None, dim=64, dtype="f32"):
    """Frame type k (a one-hot encoder frame) gives label v the logit target[v, k], whatever the decoder state:
    W_enc = identity, W_pred = 0, ReLU, so z is the one-hot frame and logits = W_out[:, k] + b_out.  Every value is a
    small dyadic number, exact in bf16 and in any summation order, so equal targets are equal logits bit for bit.
    Biases differ per label (W_out compensates), so that the tie only exists after the bias is added.
    Returns (weights, target, winners): winners[k] = lowest index among the maxima of type k (the expected argmax)."""
    blank_id = V if blank_id is None else blank_id
    NV = V + 1
    assert NV >= 300 and dim >= TIE_TYPES and blank_id in (0, V)
    lo, hi = -1.0, 2.0
    tied = [
        [3, 17],                 # two labels inside one group of 32 consecutive entries
        [3, 40],                 # same 128-entry tile, different groups of 32
        [70, 200],               # different 128-entry tiles
        [200, blank_id],         # a label and the blank
        [5, blank_id],           # a label and the blank, the label in the first tile
        [blank_id],              # blank alone: no tie
        [298],                   # one label alone: no tie
        [10, 130, 260],          # three tiles
        list(range(NV)),         # every entry equal
    ]
    target = np.full((NV, dim), lo, np.float64)
    for k, labels in enumerate(tied):
        target[labels, k] = hi
    b_out = np.array([(-0.5, 0.0, 0.25, 0.5)[v % 4] for v in range(NV)], np.float64)
    w_out = target - b_out[:, None]
    winners = [min(labels) for labels in tied]
    z = lambda *s: np.zeros(s, np.float32)
    w = dict(D=dim, E=dim, P=dim, L=1, H=dim, V=V, blank_id=blank_id, act=0, dtype=dtype, emb=z(NV, dim),
             w_ih=[z(4 * dim, dim)], w_hh=[z(4 * dim, dim)], b_ih=[z(4 * dim)], b_hh=[z(4 * dim)],
             w_enc=np.eye(dim, dtype=np.float32), b_enc=z(dim), w_pred=z(dim, dim), b_pred=z(dim),
             w_out=w_out.astype(np.float32), b_out=b_out.astype(np.float32))
    return w, target, winners


def tie_utterances(dim, types_per_utt):
    """One-hot encoder frames for lists of frame types; returns (enc [B, T, dim] zero padded, lens)."""
    T = max(len(u) for u in types_per_utt)
    enc = np.zeros((len(types_per_utt), T, dim), np.float32)
    for b, u in enumerate(types_per_utt):
        for t, k in enumerate(u):
            enc[b, t, k] = 1.0
    return enc, np.array([len(u) for u in types_per_utt], np.int32)


def tie_expected(types, winners, blank_id, S):
    """Algorithm 1 written out for the tie model: the decision on a frame never depends on the decoder, so a frame
    whose winner is a label emits it S times (the S-th emission forces the advance) and a blank frame emits nothing."""
    tok, frm = [], []
    for t, k in enumerate(types):
        if winners[k] != blank_id:
            tok += [winners[k]] * S
            frm += [t] * S
    return tok, frm
