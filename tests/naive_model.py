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
