"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU
oracle side by side on the same seeded inputs and compare everything that is
observable, element by element."""
import numpy as np
import torch

from oracle import mpe_oracle as orc
from paper_2010_11305_b200 import workloads as wl


def make_pair(cfg, tables=None, table_placement=0):
    """(Mpe handle, Oracle) for a configuration; `tables` restricts the oracle to a sample of tables."""
    from paper_2010_11305_b200 import binding as mpe
    h = mpe.Mpe(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps,
                cfg.init_lo, cfg.init_hi, cfg.seed, 0, table_placement)
    o = orc.Oracle(cfg.num_rows, cfg.dim, cfg.bits, cfg.cache_fraction, cfg.ways, cfg.policy, cfg.optimizer, cfg.eps,
                   cfg.init_lo, cfg.init_hi, cfg.seed)
    if tables is not None:
        mask = np.zeros(cfg.num_tables, np.uint8)
        mask[list(tables)] = 1
        o.set_table_mask(mask)
    return h, o


def assert_pooled_close(got, ref, abs_terms, cols=None):
    """FP32 pooled outputs: at most 1e-5 relative to the sum of absolute terms (bit-equal in practice)."""
    if cols is not None:
        got, ref, abs_terms = got[:, cols], ref[:, cols], abs_terms[:, cols]
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bound = 1e-5 * abs_terms + 1e-30
    bad = err > bound
    assert not bad.any(), f"{bad.sum()} pooled values off, worst {err.max()} vs bound {bound[bad].min()}"


def compare_state(h, o, cfg, tables, rng, n_untouched=64, check_values=True):
    """Bit-exact comparison of the low-precision entries of every row the oracle has touched plus a
    sample of untouched rows, the whole cache (tags, FP32 rows, timestamps), counters and statistics."""
    for t in tables:
        touched = o.touched(t)
        extra = rng.integers(0, cfg.num_rows[t], n_untouched)
        rows = np.unique(np.concatenate([touched, extra, [0, cfg.num_rows[t] - 1]])).astype(np.int64)
        codes, scale, bias = h.export_rows(t, rows)
        rc, rs, rb = o.rows(t, rows)
        assert np.array_equal(codes, rc), f"table {t}: codes differ on {np.nonzero((codes != rc).any(1))[0][:5]}"
        assert np.array_equal(scale.view(np.uint32), rs.view(np.uint32)), f"table {t}: scales differ"
        assert np.array_equal(bias.view(np.uint32), rb.view(np.uint32)), f"table {t}: biases differ"
        tags, crow, ts = h.export_cache(t)
        otags, ocrow, ots = o.cache(t)
        assert np.array_equal(tags, otags), f"table {t}: tags differ at {np.nonzero(tags != otags)[0][:8]}"
        if cfg.policy == wl.LRU:
            assert np.array_equal(ts, ots), f"table {t}: timestamps differ"
        if check_values:
            live = tags >= 0
            assert np.array_equal(crow[live].view(np.uint32), ocrow[live].view(np.uint32)), f"table {t}: cached rows differ"
        cnt, G = h.export_aux(t, rows)
        if cfg.policy == wl.LFU:
            assert np.array_equal(cnt, np.array([o.cnt(t, int(r)) for r in rows], np.uint32)), f"table {t}: LFU counters differ"
        if cfg.optimizer == wl.ROWWISE_ADAGRAD:
            ref = np.array([o.adagrad(t, int(r)) for r in rows], np.float32)
            assert np.array_equal(G.view(np.uint32), ref.view(np.uint32)), f"table {t}: Adagrad state differs"
        assert np.array_equal(h.stats(t), o.stats(t)), f"table {t}: stats {h.stats(t)} vs {o.stats(t)}"


def pooled_abs_terms(o, cfg, idx, off, batch, tables):
    """Sum of |fetched value| per pooled output element, from the oracle's current state (before the step)."""
    out = np.zeros((batch, cfg.num_tables * cfg.dim), np.float64)
    d = cfg.dim
    for t in tables:
        cache = {}
        for b in range(batch):
            bag = t * batch + b
            for p in range(off[bag], off[bag + 1]):
                r = int(idx[p])
                if r < 0 or r >= cfg.num_rows[t]:
                    continue
                if r not in cache:
                    cache[r] = np.abs(o.fetch_value(t, r)).astype(np.float64)
                out[b, t * d:(t + 1) * d] += cache[r]
    return out


def run_parity(cfg, steps, tables=None, stream_device="cpu", check_every=1, abs_terms_steps=1, seed=0):
    """Run `steps` training steps on both sides and compare after every `check_every` steps."""
    all_tables = list(range(cfg.num_tables)) if tables is None else list(tables)
    h, o = make_pair(cfg, tables)
    st = wl.Stream(cfg, stream_device)
    rng = np.random.default_rng(seed)
    dev = torch.device("cuda:0")
    cols = np.concatenate([np.arange(t * cfg.dim, (t + 1) * cfg.dim) for t in all_tables])
    compare_state(h, o, cfg, all_tables, rng)           # initial tables
    info = []
    for step in range(1, steps + 1):
        idx, off, grad = st.batch(step)
        d_idx, d_off, d_grad = idx.to(dev), off.to(dev), grad.to(dev)
        d_out = torch.empty(cfg.batch, cfg.num_tables * cfg.dim, dtype=torch.float32, device=dev)
        idx_h, off_h, grad_h = idx.cpu().numpy(), off.cpu().numpy(), grad.cpu().numpy()
        h.forward(d_idx, d_off, cfg.batch, d_out)
        ref = o.forward(idx_h, off_h, cfg.batch)
        got = d_out.cpu().numpy()
        if step <= abs_terms_steps and idx_h.size <= 200_000:
            assert_pooled_close(got, ref, pooled_abs_terms(o, cfg, idx_h, off_h, cfg.batch, all_tables), cols)
        assert np.array_equal(got[:, cols], ref[:, cols]), f"step {step}: pooled outputs are not bit-equal"
        h.backward(d_grad, cfg.lr, step)
        o.backward(grad_h, cfg.lr, step)
        code, detail = h.last_error()
        assert code == 0, (code, detail)
        info.append(h.step_info())
        if step % check_every == 0 or step == steps:
            compare_state(h, o, cfg, all_tables, rng)
    h.flush()
    o.flush()
    compare_state(h, o, cfg, all_tables, rng)
    return h, o, info
