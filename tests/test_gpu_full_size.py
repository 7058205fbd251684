"""Parity at the benchmark's full sizes (configurations 3-5 and two of the small-suffix shapes), in the
launch configuration the benchmark times: the layer-dispatch call at selected layers, compared with the oracle on sampled
rows, each computed over all of its keys.  Sampled per layer: tile-boundary rows of the shortest and
longest requests and random (request, head, row) triples."""
import numpy as np
import pytest
import torch

import oracle
import __graft_entry__ as entry
from paper_2606_07571_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def run_config(name, layers_to_check, n_random=24, key_ranges=False):
    entry.build()
    w = workloads.CONFIGS[name]()
    L = w.num_layers
    npages = w.pages_needed() + 1
    order = workloads.shuffled_page_order(npages, 7) if w.shuffle_pages else None
    bc = binding.BiCache(L, w.num_q_heads, w.num_kv_heads, w.head_dim, npages, w.dtype, w.total_rows,
                         w.num_requests, free_order=order)
    table = workloads.standin_depth_table(L)
    bc.set_depth_table(table)
    # the oracle's store holds only the checked layers (its layer j = layers_to_check[j])
    st = oracle.PagedPrefixStore(len(layers_to_check), w.num_kv_heads, w.head_dim, 16, npages, free_order=order)
    pid, opid = [], []
    for g in range(len(w.prefix_lens)):
        kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
        p, hit, pages = bc.put_prefix(workloads.prefix_key(w, g), kc, vc)
        op, _, opages = st.put(workloads.prefix_key(w, g), workloads.to_f64(kc[layers_to_check]),
                               workloads.to_f64(vc[layers_to_check]))
        assert (p, pages) == (op, opages) and not hit                     # ids and page lists bit-exact
        pid.append(p)
        opid.append(op)
        del kc, vc
    depth = bc.reuse_depth(w.req_prefix_len(), w.suffix_lens)
    assert (depth == oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, table, L)).all()
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    out = torch.empty_like(q)
    lse = torch.empty(q.shape[:2], dtype=torch.float32, device="cuda")
    req_pid = [pid[g] for g in w.req_prefix]
    rng = np.random.default_rng(5)
    by_len = np.argsort(w.suffix_lens)
    picked = sorted({int(by_len[0]), int(by_len[-1]), int(by_len[len(by_len) // 2])} |
                    {int(x) for x in rng.integers(0, w.num_requests, 3)})
    heads = sorted({0, w.num_q_heads - 1, int(rng.integers(w.num_q_heads))})
    for lp, layer in enumerate(layers_to_check):
        out.fill_(7.0)
        bc.attend_layer(layer, depth, req_pid, w.full_row_off, w.full_lens, q, k, v, out, lse, w.softmax_scale)
        assert bc.device_status() == binding.OK
        if key_ranges and layer < int(min(depth)):
            # every request reuses at this layer: one attend call, served by the key-range kernel
            assert bc.last_attention_kernel() == binding.KERNEL_KEY_RANGES
        worst = 0.0
        errs = []
        for i in picked:
            off, N, m = w.full_row_off[i], w.full_lens[i], w.prefix_lens[w.req_prefix[i]]
            n = N - m
            qi, ki, vi = (workloads.to_f64(x[off:off + N]) for x in (q, k, v))
            got = workloads.to_f64(out[off:off + N])
            got_lse = workloads.to_f64(lse[off:off + N])
            reuse = layer < depth[i]
            if reuse:
                rows = sorted({0, 63, 64, 127, 128, 255, 256, n - 1} & set(range(n)) |
                              {int(x) for x in rng.integers(0, n, n_random // 4)})
                samples = [(0, h, a) for a in rows for h in heads]
                ref, ref_lse = oracle.attend_rows(st, lp, [opid[w.req_prefix[i]]], [m], [n], qi, ki, vi,
                                                  w.softmax_scale, samples)
                got_rows = np.stack([got[m + a, h] for _, h, a in samples])
                got_l = np.array([got_lse[m + a, h] for _, h, a in samples])
                assert (got[:m] == 7.0).all()                               # prefix rows are not produced
            else:
                rows = sorted({0, 127, 128, m - 1, m, m + 1, N - 1} & set(range(N)) |
                              {int(x) for x in rng.integers(0, N, n_random // 4)})
                samples = [(0, h, a) for a in rows for h in heads]
                ref, ref_lse = oracle.attend_full_rows([0], [N], qi, ki, vi, w.softmax_scale, samples)
                got_rows = np.stack([got[a, h] for _, h, a in samples])
                got_l = np.array([got_lse[a, h] for _, h, a in samples])
            err = np.abs(got_rows - ref)
            assert np.isfinite(got_rows).all()
            assert err.max() <= 2e-2, "%s layer %d request %d: max|err| %.4g" % (name, layer, i, err.max())
            assert np.abs(got_l - ref_lse).max() <= 1e-3
            errs.append(err.mean())
            worst = max(worst, err.max())
        assert np.mean(errs) <= 2e-3
    bc.close()
    return depth


def test_config3_full_size_sampled():
    w = workloads.config3()
    d = oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, workloads.standin_depth_table(32), 32)
    run_config("config3", sorted({0, int(d.min()) - 1, int(d.min()), int(np.median(d)), 31}))


def test_config4_full_size_sampled():
    w = workloads.config4()
    d = oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, workloads.standin_depth_table(32), 32)
    run_config("config4", sorted({0, int(np.median(d)), 31}))


def test_config5_full_size_sampled():
    run_config("config5", [0, 20, 21])          # depth is 21 for every request: last reuse layer, first full layer


@pytest.mark.parametrize("name", ["b2", "b3"])
def test_small_suffix_shapes_full_size_sampled(name):
    """Block-query shapes at full size (prefix 16384, 1 and 4 requests of 32 tokens, 32 layers): the
    shallow layers go through the key-range kernel, the deep ones through full attention."""
    w = workloads.CONFIGS[name]()
    d = oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, workloads.standin_depth_table(w.num_layers),
                           w.num_layers)
    run_config(name, sorted({0, int(d.min()) - 1, int(d.min())}), key_ranges=True)
