"""An independent dense statement of the SDQ decomposition used ONLY to pin the oracle.

It never builds packed arrays: it computes masks and quantized dense matrices directly with
vectorised numpy, threshold-based E2M1 rounding and torch's own float8_e4m3fn cast, i.e. with none
of the oracle's routines.
"""
import numpy as np
import torch

E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def bf16_to_f64(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()


def q_e2m1(v):
    """round |v| to the E2M1 grid, ties to the neighbour with even code, saturate at 6; keeps sign."""
    a = np.abs(v)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    tie_up = np.array([False, True, False, True, False, True, False])
    code = np.zeros(a.shape, dtype=np.int64)
    for i in range(7):
        code = np.where((a > mids[i]) | ((a == mids[i]) & tie_up[i]), i + 1, code)
    return np.copysign(E2M1_VALUES[code], v)


def q_e4m3(v):
    t = torch.from_numpy(np.ascontiguousarray(v)).to(torch.float32)
    assert (t.abs() <= 448).all()
    return t.to(torch.float8_e4m3fn).double().numpy()


def floor_log2(a):
    m, e = np.frexp(a)          # a = m * 2^e, m in [0.5, 1)
    return e - 1


def ceil_exp(amax, vmax):
    """smallest integer e with amax <= vmax * 2^e (amax > 0)"""
    e = np.ceil(np.log2(amax / vmax)).astype(np.int64)
    e = np.where(amax > np.ldexp(vmax, e), e + 1, e)
    e = np.where(amax <= np.ldexp(vmax, e - 1), e - 1, e)
    return e


def block_scale_exp(amax, rule_floor):
    E = np.where(amax > 0, floor_log2(np.where(amax > 0, amax, 1.0)) - 2 if rule_floor
                 else ceil_exp(np.where(amax > 0, amax, 1.0), 6.0), -127)
    return np.clip(E, -127, 127)


def top_mask(keys, n):
    """mask of the n largest along the last axis, ties to the lower index"""
    order = np.argsort(-keys, axis=-1, kind="stable")
    mask = np.zeros(keys.shape, dtype=bool)
    np.put_along_axis(mask, order[..., :n], True, axis=-1)
    return mask


def decompose_dense(W_bits, out_n, pair, block, rule_floor, col_weight=None, small=False):
    """returns (W_in_hat, W_out_hat, mask_in_slots, mask_out) as dense [N, K] arrays; with col_weight the
    selections rank by the fp32 product |w| * c[k] instead of |w| (the values that get quantized do not change);
    rule_floor: True = OCP floor rule, False = ceil rule, "ue4m3" = two-level scaling with e4m3 scales;
    pair: True = pair-wise 4:8, False = element-wise 2:4, None = no pruning,
    an integer n = the n most significant of every 8 survive (outliers included)"""
    W = bf16_to_f64(W_bits)
    N, K = W.shape
    A = np.abs(W)
    if col_weight is not None:
        A = (A.astype(np.float32) * np.asarray(col_weight, dtype=np.float32)[None, :]).astype(np.float32).astype(np.float64)
    Ao = -A if small else A               # "Small": the least significant values become the outliers
    if pair == "3of4":                    # S-Vectors of 4: the largest of every 4 is the outlier, the next two stay
        mask_out = top_mask(Ao.reshape(N, K // 4, 4), 1).reshape(N, K) if out_n else np.zeros((N, K), bool)
    else:
        mask_out = top_mask(Ao.reshape(N, K // 8, 8), out_n).reshape(N, K) if out_n else np.zeros((N, K), bool)
    R = np.where(mask_out, 0.0, A)
    if pair == "3of4":
        keys = np.where(mask_out, -1.0, A).reshape(N, K // 4, 4)
        slots = top_mask(keys, 3 - (1 if out_n else 0)).reshape(N, K)
    elif pair is None:                      # no pruning: every non-outlier value stays an inlier
        slots = np.ones((N, K), bool)
    elif pair is not True and pair is not False:   # an integer n: keep the n most significant of every 8 in total
        keys = np.where(mask_out, -1.0, A).reshape(N, K // 8, 8)
        slots = top_mask(keys, int(pair) - out_n).reshape(N, K)
    elif pair:
        r32 = R.astype(np.float32).reshape(N, K // 8, 4, 2)
        score = (r32[..., 0] + r32[..., 1]).astype(np.float32)
        keep_pair = top_mask(score, 2)
        slots = np.repeat(keep_pair, 2, axis=-1).reshape(N, K)
    else:
        keys = np.where(mask_out, -1.0, A).reshape(N, K // 4, 4)
        slots = top_mask(keys, 2).reshape(N, K)
    inl = slots & ~mask_out
    Win = np.where(inl, W, 0.0)
    if rule_floor == "ue4m3":
        Win_hat, _ = two_level_quantize(Win, inl, block)
    else:
        amax = np.abs(Win).reshape(N, K // block, block).max(-1)
        E = block_scale_exp(amax, rule_floor)
        Es = np.repeat(E, block, axis=1)
        Win_hat = np.where(inl, np.ldexp(q_e2m1(np.ldexp(Win, -Es)), Es), 0.0)
    Wout = np.where(mask_out, W, 0.0)
    oamax = np.abs(Wout).max(axis=1)
    e = np.where(oamax > 0, ceil_exp(np.where(oamax > 0, oamax, 1.0), 448.0), 0)[:, None]
    Wout_hat = np.ldexp(q_e4m3(np.ldexp(Wout, -e)), e)
    return Win_hat, Wout_hat, slots, mask_out


def quantize_act_dense(X_bits, block, rule_floor):
    X = bf16_to_f64(X_bits)
    M, K = X.shape
    if rule_floor == "ue4m3":
        A_i, _ = two_level_quantize(X, np.ones(X.shape, bool), block)
    else:
        amax = np.abs(X).reshape(M, K // block, block).max(-1)
        Es = np.repeat(block_scale_exp(amax, rule_floor), block, axis=1)
        A_i = np.ldexp(q_e2m1(np.ldexp(X, -Es)), Es)
    ramax = np.abs(X).max(axis=1)
    e = np.where(ramax > 0, ceil_exp(np.where(ramax > 0, ramax, 1.0), 448.0), 0)[:, None]
    A_o = np.ldexp(q_e4m3(np.ldexp(X, -e)), e)
    return A_i, A_o


def two_level_quantize(V, counted, block):
    """Two-level scaling with fp8-e4m3 Q-Vector scales, stated with numpy and torch's own float8 cast: per row a
    power-of-two factor 2^t (smallest t with amax <= 448 * 2^t over the counted elements), per block the e4m3 value
    nearest to amax_b / (6 * 2^t) (at least 2^-9 unless the block is all zero), per element the E2M1 value nearest
    to v / scale.  V [R, K] fp64, counted [R, K] bool (elements that exist); returns the dequantized values."""
    R, K = V.shape
    A = np.where(counted, np.abs(V), 0.0)
    ramax = A.max(axis=1)
    t = np.where(ramax > 0, ceil_exp(np.where(ramax > 0, ramax, 1.0), 448.0), 0)[:, None]
    bamax = A.reshape(R, K // block, block).max(-1)
    y = np.ldexp(bamax, -t) / 6.0
    s = torch.from_numpy(y.astype(np.float32)).to(torch.float8_e4m3fn).double().numpy()
    s = np.where((bamax > 0) & (s == 0), 2.0 ** -9, s)
    S = np.repeat(np.ldexp(s, t), block, axis=1)
    q = np.where(S > 0, V / np.where(S > 0, S, 1.0), 0.0)
    return np.where(counted, q_e2m1(q) * S, 0.0), t[:, 0]
