"""Why the workload with a smooth low-frequency component is compared stage by stage when its
summary projections are the identity: shown with the fp64 oracle alone, no GPU.

With U = I the low band's summary tokens are as large as its coefficients (a separable cosine of
amplitude 3 puts 3 sqrt(N / 8) into one coefficient), the summary logits of the mid and high bands'
tokens reach several hundred, and the softmax over the 2m summaries sits on near-ties between huge
logits: rounding a band token to bf16 -- a change of at most 0.016 -- then moves its exchanged value
by tens and the layer's output by far more than the tolerance.  With summary projections scaled so
that the logits are of order one the same rounding moves the output by less than half the
tolerance; that variant is what the GPU tests compare end to end."""
import numpy as np

from oracle import freqformer_oracle as O
from paper_2604_22808_b200 import configs as C
from paper_2604_22808_b200 import inputs as I

WELL_CONDITIONED_U_SCALE = 1.0 / 256.0


def _rounding_sensitivity(cfg, U):
    """Largest logit, and how far the output of one head moves when the mid- and high-band tokens
    that enter the exchange are rounded to bf16 (their storage type on the device)."""
    Q, K, V = (I.qkv_full(cfg, t)[0] for t in range(3))
    res = O.forward_sample(cfg, Q, K, V, I.router_weights(cfg), U, cfg.timesteps[0],
                           alloc=[0] * cfg.heads, want_taps=True)          # pass-through: Y = V~
    members = O.band_members(cfg.grid, cfg.low_cut, cfg.mid_cut)
    d = cfg.head_dim
    Y, S = res["taps"]["Y"][0], res["taps"]["S"][0]
    exact, rounded = np.zeros((cfg.N, d)), np.zeros((cfg.N, d))
    logit_max = token_move = 0.0
    for l in range(3):
        Z = np.concatenate([S[o] for o in range(3) if o != l])
        Yr = Y[l] if l == 0 else I.round_to_bf16(Y[l].astype(np.float32)).astype(np.float64)
        assert np.abs(Yr - Y[l]).max() <= 0.016
        a, b = O.exchange(Y[l], Z), O.exchange(Yr, Z)
        logit_max = max(logit_max, float(np.abs(Y[l] @ Z.T).max() / np.sqrt(d)))
        token_move = max(token_move, float(np.abs(a - b).max()))
        exact[members[l]], rounded[members[l]] = a, b
    shape = (cfg.T, cfg.H, cfg.W, d)
    out_move = float(np.abs(O.inverse_transform(exact.reshape(shape)) - O.inverse_transform(rounded.reshape(shape))).max())
    return logit_max, token_move, out_move


def test_smooth_workload_with_identity_summaries_is_ill_conditioned():
    cfg = C.R256K.scaled("256k_replica_1head", heads=1)
    logit_max, token_move, out_move = _rounding_sensitivity(cfg, I.summary_projection(cfg))
    assert logit_max > 100.0
    assert token_move > 1.0            # a 0.016 rounding of a token becomes an O(10) change of its exchanged value
    assert out_move > 10 * 2e-2        # ... and the output moves by far more than the tolerance


def test_smooth_workload_with_scaled_summaries_is_well_conditioned():
    cfg = C.R256K.scaled("256k_replica_1head", heads=1)
    U = I.summary_projection(cfg, identity=False, scale=WELL_CONDITIONED_U_SCALE)
    logit_max, token_move, out_move = _rounding_sensitivity(cfg, U)
    assert logit_max < 8.0
    assert token_move < 2e-2 and out_move < 1e-2
