"""Glue between the seeded workloads, the CPU oracle and the CUDA path for the parity tests."""
import numpy as np

from paper_2402_11131_b200 import workloads as W

MAX_ABS_TOL = 2e-2     # attention output, unit-variance bf16 V, fp32 accumulation
MEAN_ABS_TOL = 2e-3
LSE_TOL = 2e-3       # log-sum-exp in fp32: the row sums are taken before the weights are rounded to bf16


def oracle_layer(oracle, st, ly, b, node_sel=None, heads=None):
    """Oracle attention of sequence b for one layer's host tensors."""
    T = st.nodes(b)
    s0 = int(st.kv_start[b])
    cap = int(st.kv_capacity[b])
    g = st.cfg.gamma if ly.is_msa else 0
    sel = None if node_sel is None else np.ascontiguousarray(node_sel[:T], dtype=np.uint8)
    return oracle.msa_attention(
        st.parent[b][:T], int(st.kv_len[b]), g, st.sm_scale, ly.q_main[b][:T], ly.k_cache[s0:s0 + cap],
        ly.v_cache[s0:s0 + cap], None if g == 0 else ly.q_spec[b][:T], None if g == 0 else ly.k_spec[b][:T],
        None if g == 0 else ly.v_spec[b][:T], node_sel=sel, heads=heads)


def compare_attention(oracle, st, ly, dev, i, seqs=None, node_sel=None, heads=None, check_lse=False):
    """Compares layer slot i of DeviceStep `dev` with the oracle.  Returns (max_abs, mean_abs, n)."""
    from paper_2402_11131_b200 import api
    o_main = W.bf16_bits_to_f64(api.bf16_to_host_bits(dev.o_main[i]))
    o_spec = None if not ly.is_msa else W.bf16_bits_to_f64(api.bf16_to_host_bits(dev.o_spec[i]))
    errs = []
    lse_err = 0.0
    for b in (range(st.cfg.batch) if seqs is None else seqs):
        T = st.nodes(b)
        om, lm, os_, ls = oracle_layer(oracle, st, ly, b, node_sel, heads)
        mask = ~np.isnan(om)
        assert mask.any()
        errs.append(np.abs(o_main[b][:T][mask] - om[mask]))
        if ly.is_msa:
            mask_s = ~np.isnan(os_)
            errs.append(np.abs(o_spec[b][:T][mask_s] - os_[mask_s]))
        if check_lse:
            lg = dev.lse_main[i][b][:T].double().cpu().numpy()
            mk = ~np.isnan(lm)
            lse_err = max(lse_err, float(np.abs(lg[mk] - lm[mk]).max()))
            if ly.is_msa:
                lg = dev.lse_spec[i][b][:T].double().cpu().numpy()
                mk = ~np.isnan(ls)
                lse_err = max(lse_err, float(np.abs(lg[mk] - ls[mk]).max()))
    e = np.concatenate([x.ravel() for x in errs])
    assert np.isfinite(e).all(), "non-finite attention output"
    return float(e.max()), float(e.mean()), int(e.size), lse_err


def assert_attention_close(oracle, st, ly, dev, i, **kw):
    mx, mean, n, lse_err = compare_attention(oracle, st, ly, dev, i, **kw)
    assert mx <= MAX_ABS_TOL and mean <= MEAN_ABS_TOL, (mx, mean, n)
    if kw.get("check_lse"):
        assert lse_err <= LSE_TOL, lse_err
    return mx, mean
