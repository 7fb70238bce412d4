"""fp64 oracle of the attention score layer (Section 4.1, the score equation and the arg max).

TEST INFRASTRUCTURE ONLY: plain numpy, no code shared with the CUDA library.

    score_t = W^score Mean(X_[t])        one score per operation, chunk and head
    opt_t   = arg max softmax(score_t)   the operation assigned to chunk t

X [B, L, d_model]; W^score [H, 2, d_model] (operation 0 = linear attention, 1 = softmax attention;
every head has its own pair of rows: "each linear attention head receives its own mask",
Section 4.3).  Returns scores [B, L/C, H, 2] and route [B, L, H] uint8 (1 = softmax), the chunk's
decision repeated over its C tokens.  The softmax is monotone, so the arg max is taken on the
scores; on a tie the first operation (linear) wins, as numpy's argmax does.
"""
import numpy as np


def score_layer(x, w_score, C=64):
    x = np.asarray(x, np.float64)
    w_score = np.asarray(w_score, np.float64)
    B, L, Dm = x.shape
    H = w_score.shape[0]
    assert w_score.shape == (H, 2, Dm) and L % C == 0
    pooled = x.reshape(B, L // C, C, Dm).mean(axis=2)              # Mean over the chunk's tokens
    scores = np.einsum("bcd,hod->bcho", pooled, w_score)
    opt = np.argmax(scores, axis=-1).astype(np.uint8)              # [B, L/C, H]
    route = np.repeat(opt, C, axis=1)
    return dict(scores=scores, route=route)
