"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle on the same
seeded inputs.  Tolerances: bf16 outputs max-abs 2e-2 and mean-abs 2e-3, fp32 outputs 1e-4;
log-sum-exp 1e-3 (bf16 inputs) / 1e-5 (fp32); depths and page indices bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import __graft_entry__ as entry
from paper_2606_07571_b200 import binding, workloads

pytestmark = pytest.mark.gpu

TOL = {torch.bfloat16: (2e-2, 2e-3, 1e-3), torch.float32: (1e-4, 1e-5, 1e-5)}


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    binding.load_library()


def check(got, ref, dtype, what):
    max_tol, mean_tol, _ = TOL[dtype]
    err = np.abs(got - ref)
    assert np.isfinite(got).all(), what + ": non-finite output"
    assert err.max() <= max_tol, "%s: max|err| %.4g > %.4g" % (what, err.max(), max_tol)
    assert err.mean() <= mean_tol, "%s: mean|err| %.4g > %.4g" % (what, err.mean(), mean_tol)


class Case:
    """Device context + oracle store filled with the same prefixes."""

    def __init__(self, w, path=binding.PATH_AUTO, extra_pages=1, layers=None, device_gen=False):
        self.w = w
        npages = w.pages_needed() + extra_pages
        order = workloads.shuffled_page_order(npages, 7) if w.shuffle_pages else None
        self.bc = binding.BiCache(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, npages, w.dtype,
                                  w.total_rows, w.num_requests, free_order=order)
        self.bc.set_path(path)
        table = workloads.standin_depth_table(w.num_layers)
        self.bc.set_depth_table(table)
        self.layers = list(range(w.num_layers)) if layers is None else layers
        # the oracle keeps only the layers that are checked (layer j of its store = self.layers[j])
        self.st = oracle.PagedPrefixStore(len(self.layers), w.num_kv_heads, w.head_dim, 16, npages, free_order=order)
        self.pid, self.opid = [], []
        for g in range(len(w.prefix_lens)):
            kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
            pid, hit, pages = self.bc.put_prefix(workloads.prefix_key(w, g), kc, vc)
            opid, ohit, opages = self.st.put(workloads.prefix_key(w, g), workloads.to_f64(kc[self.layers]),
                                             workloads.to_f64(vc[self.layers]))
            assert (pid, hit, pages) == (opid, ohit, opages)
            assert self.bc.prefix_pages(pid) == opages
            self.pid.append(pid)
            self.opid.append(opid)
        depth = self.bc.reuse_depth(w.req_prefix_len(), w.suffix_lens)
        self.depth = oracle.reuse_depth(w.req_prefix_len(), w.suffix_lens, table, w.num_layers)
        assert (depth == self.depth).all()
        self.q, self.k, self.v = workloads.draw_full_qkv(w, "cuda")
        self.req_pid = [self.pid[g] for g in w.req_prefix]
        self.req_opid = [self.opid[g] for g in w.req_prefix]

    def host(self):
        return tuple(workloads.to_f64(x) for x in (self.q, self.k, self.v))

    def run_attend(self, layer, reqs=None):
        w = self.w
        reqs = list(range(w.num_requests)) if reqs is None else reqs
        out = torch.full_like(self.q, 7.0)
        lse = torch.full(self.q.shape[:2], 7.0, dtype=torch.float32, device="cuda")
        self.bc.attend(layer, [self.req_pid[i] for i in reqs], [w.suffix_row_off[i] for i in reqs],
                       [w.suffix_lens[i] for i in reqs], self.q, self.k, self.v, out, lse, w.softmax_scale)
        assert self.bc.device_status() == binding.OK
        return out, lse

    def run_full(self, layer, reqs=None):
        w = self.w
        reqs = list(range(w.num_requests)) if reqs is None else reqs
        out = torch.full_like(self.q, 7.0)
        lse = torch.full(self.q.shape[:2], 7.0, dtype=torch.float32, device="cuda")
        self.bc.attend_full(layer, [w.full_row_off[i] for i in reqs], [w.full_lens[i] for i in reqs],
                            self.q, self.k, self.v, out, lse, w.softmax_scale)
        assert self.bc.device_status() == binding.OK
        return out, lse

    def compare_all(self, layer_pos=0, full=True):
        """Element-by-element comparison of one layer (attend on every request, then attend_full)."""
        w = self.w
        layer = self.layers[layer_pos]
        qd, kd, vd = self.host()
        out, lse = self.run_attend(layer)
        ref, ref_lse = oracle.attend(self.st, layer_pos, self.req_opid, w.suffix_row_off, w.suffix_lens,
                                     qd, kd, vd, w.softmax_scale)
        got, got_lse = workloads.to_f64(out), workloads.to_f64(lse)
        mask = np.zeros(w.total_rows, dtype=bool)
        for o, n in zip(w.suffix_row_off, w.suffix_lens):
            mask[o:o + n] = True
        check(got[mask], ref[mask], w.dtype, w.name + " attend")
        assert np.abs(got_lse[mask] - ref_lse[mask]).max() <= TOL[w.dtype][2]
        assert (got[~mask] == 7.0).all() and (got_lse[~mask] == 7.0).all()      # untouched rows
        if full:
            out, lse = self.run_full(layer)
            ref, ref_lse = oracle.attend_full(w.full_row_off, w.full_lens, qd, kd, vd, w.softmax_scale)
            check(workloads.to_f64(out), ref, w.dtype, w.name + " attend_full")
            assert np.abs(workloads.to_f64(lse) - ref_lse).max() <= TOL[w.dtype][2]

    def close(self):
        self.bc.close()


def tiny(name, L, Hq, Hkv, D, dtype, ms, req_prefix, ns, shuffle=False, std=1.0, scale=None):
    return workloads.Workload(name, L, Hq, Hkv, D, dtype, 16, ms, req_prefix, ns,
                              softmax_scale=(D ** -0.5 if scale is None else scale), value_std=std,
                              shuffle_pages=shuffle)


def test_config1_tiny_fp32():
    c = Case(workloads.config1())
    c.compare_all()
    assert c.bc.last_attention_kernel() == binding.KERNEL_SIMT      # fp32, D = 64: the CUDA-core kernel
    c.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shape", [
    (2, 4, 2, 64, [70, 5], [0, 0, 1], [33, 1, 40]),
    (1, 6, 3, 32, [17], [0, 0], [0, 9]),
    (2, 2, 2, 128, [130, 16, 33], [0, 1, 1, 2], [5, 129, 31, 64]),
    (1, 8, 2, 128, [257], [0], [77]),
])
def test_random_small_shapes_simt(dtype, shape):
    L, Hq, Hkv, D, ms, rp, ns = shape
    c = Case(tiny("small", L, Hq, Hkv, D, dtype, ms, rp, ns, shuffle=True), path=binding.PATH_SIMT)
    for lp in range(L):
        c.compare_all(lp)
    c.close()


def test_peaked_logits_and_partial_pages():
    """Large scores (the running maximum moves a lot, in the prefix, the suffix and the last
    partial page) must not break the rescaling."""
    for scale in (0.5, 1.0):
        c = Case(tiny("peaked", 1, 4, 2, 128, torch.bfloat16, [203], [0, 0], [150, 37], std=1.0, scale=scale))
        c.compare_all()
        c.close()


def test_no_prefix_equals_full_and_empty_requests():
    w = tiny("noprefix", 1, 4, 4, 128, torch.bfloat16, [48], [0, 0, 0], [0, 130, 20])
    c = Case(w)
    out, lse = c.run_attend(0)                                   # with prefix, includes an empty request
    # prefix_id = -1: attend degenerates to attention over the suffix alone = attend_full on those rows
    o1 = torch.zeros_like(c.q)
    c.bc.attend(0, [-1, -1, -1], w.suffix_row_off, w.suffix_lens, c.q, c.k, c.v, o1, None, w.softmax_scale)
    o2 = torch.zeros_like(c.q)
    c.bc.attend_full(0, w.suffix_row_off, w.suffix_lens, c.q, c.k, c.v, o2, None, w.softmax_scale)
    assert c.bc.device_status() == binding.OK
    assert torch.equal(o1, o2)
    qd, kd, vd = c.host()
    ref, _ = oracle.attend(c.st, 0, [-1] * 3, w.suffix_row_off, w.suffix_lens, qd, kd, vd, w.softmax_scale)
    rows = np.concatenate([np.arange(o, o + n) for o, n in zip(w.suffix_row_off, w.suffix_lens)])
    check(workloads.to_f64(o1)[rows], ref[rows], w.dtype, "no prefix")
    # all-empty batch and R = 0 are legal no-ops
    c.bc.attend(0, [c.pid[0]], [0], [0], c.q, c.k, c.v, o1, None, w.softmax_scale)
    c.bc.attend(0, [], [], [], c.q, c.k, c.v, o1, None, w.softmax_scale)
    c.close()


def test_subset_dispatch_and_strided_rows():
    """A layer's reuse set and full set are subsets of the batch; q may have a larger row stride."""
    w = tiny("subset", 2, 4, 2, 128, torch.bfloat16, [90, 40], [0, 0, 1, 1], [20, 140, 7, 64])
    c = Case(w)
    qd, kd, vd = c.host()
    big = torch.zeros(w.total_rows, 2 * w.num_q_heads, w.head_dim, dtype=w.dtype, device="cuda")
    big[:, :w.num_q_heads] = c.q
    c.q = big[:, :w.num_q_heads]                                  # row stride 2*Hq*D
    reuse, full = [1, 2], [0, 3]
    out, lse = c.run_attend(1, reuse)
    ref, _ = oracle.attend(c.st, 1, [c.req_opid[i] for i in reuse], [w.suffix_row_off[i] for i in reuse],
                           [w.suffix_lens[i] for i in reuse], qd, kd, vd, w.softmax_scale)
    rows = np.concatenate([np.arange(w.suffix_row_off[i], w.suffix_row_off[i] + w.suffix_lens[i]) for i in reuse])
    check(workloads.to_f64(out)[rows], ref[rows], w.dtype, "reuse subset")
    out, lse = c.run_full(1, full)
    ref, _ = oracle.attend_full([w.full_row_off[i] for i in full], [w.full_lens[i] for i in full],
                                qd, kd, vd, w.softmax_scale)
    rows = np.concatenate([np.arange(w.full_row_off[i], w.full_row_off[i] + w.full_lens[i]) for i in full])
    check(workloads.to_f64(out)[rows], ref[rows], w.dtype, "full subset")
    c.close()


def test_stack_dispatch_matches_oracle_stack():
    """One denoising step: per-request depths from the rule, layer l reuses iff l < depth."""
    w = tiny("stack", 4, 4, 2, 128, torch.bfloat16, [200, 24], [0, 0, 1], [30, 150, 100])
    c = Case(w)
    depth = [1, 4, 0]                                               # mixed; also exercises 0 and L
    qd, kd, vd = c.host()
    ref = oracle.stack(c.st, depth, c.req_opid, w.req_prefix_len(), w.full_row_off, w.full_lens,
                       [qd] * 4, [kd] * 4, [vd] * 4, w.softmax_scale)
    for l in range(4):
        out = torch.zeros_like(c.q)
        lse = torch.full(c.q.shape[:2], -float("inf"), dtype=torch.float32, device="cuda")
        reuse = [i for i in range(3) if l < depth[i]]
        full = [i for i in range(3) if l >= depth[i]]
        if reuse:
            c.bc.attend(l, [c.req_pid[i] for i in reuse], [w.suffix_row_off[i] for i in reuse],
                        [w.suffix_lens[i] for i in reuse], c.q, c.k, c.v, out, lse, w.softmax_scale)
        if full:
            c.bc.attend_full(l, [w.full_row_off[i] for i in full], [w.full_lens[i] for i in full],
                             c.q, c.k, c.v, out, lse, w.softmax_scale)
        assert c.bc.device_status() == binding.OK
        check(workloads.to_f64(out), ref[l][0], w.dtype, "stack layer %d" % l)
        got_lse = workloads.to_f64(lse)
        fin = np.isfinite(ref[l][1])
        assert (np.isfinite(got_lse) == fin).all()
        assert np.abs(got_lse[fin] - ref[l][1][fin]).max() <= 1e-3
    c.close()


def test_key_split_path_small_suffix():
    """Few query rows over a long prefix: keys are split across CTAs and merged."""
    w = workloads.scaled_down(workloads.small_suffix("b3"), num_layers=1, prefix_div=4)     # m=4096, 4 x 32 rows
    c = Case(w)
    c.compare_all(full=False)
    c.close()
    w = tiny("split-gqa", 1, 28, 4, 128, torch.bfloat16, [3000], [0], [16])
    c = Case(w)
    c.compare_all(full=False)
    c.close()


def test_eviction_then_reput_and_status_codes():
    w = tiny("evict", 1, 2, 2, 128, torch.bfloat16, [40, 40], [0, 1], [8, 8])
    c = Case(w, extra_pages=0)                                      # pool exactly full: 3 + 3 pages
    kc, vc = workloads.draw_prefix_kv(w, 0, "cuda")
    new_pid, hit, pages = c.bc.put_prefix(999, kc[:, :33], vc[:, :33])      # evicts prefix 0 (oldest)
    assert not hit and new_pid == 2 and pages == c.st.put(999, workloads.to_f64(kc[:, :33]),
                                                          workloads.to_f64(vc[:, :33]))[2]
    out = torch.zeros_like(c.q)
    with pytest.raises(binding.BiCacheError) as e:
        c.bc.attend(0, [c.pid[0]], [0], [4], c.q, c.k, c.v, out)
    assert e.value.status == binding.ERR_NOTFOUND
    with pytest.raises(binding.BiCacheError) as e:
        c.bc.attend(0, [c.pid[1], new_pid, c.pid[1]], [0, 8, 16], [4, 4, 4], c.q, c.k, c.v, out)
    assert e.value.status == binding.ERR_INVALID                    # ids not contiguous
    with pytest.raises(binding.BiCacheError) as e:
        c.bc.attend(3, [new_pid], [0], [4], c.q, c.k, c.v, out)
    assert e.value.status == binding.ERR_INVALID                    # layer out of range
    with pytest.raises(binding.BiCacheError) as e:
        c.bc.attend_full(0, [0], [-1], c.q, c.k, c.v, out)
    assert e.value.status == binding.ERR_INVALID
    assert (out == 0).all()                                         # errors leave outputs untouched
    # the evicted-and-replaced prefix is served correctly from its new pages
    qd, kd, vd = c.host()
    c.bc.attend(0, [new_pid], [0], [8], c.q, c.k, c.v, out, None, w.softmax_scale)
    ref, _ = oracle.attend(c.st, 0, [2], [0], [8], qd, kd, vd, w.softmax_scale)
    check(workloads.to_f64(out)[:8], ref[:8], w.dtype, "after eviction")
    c.close()


def test_config2_attend_complete_and_full_sampled():
    w = workloads.config2()
    c = Case(w)
    c.compare_all(full=False)
    out, lse = c.run_full(0)
    rng = np.random.default_rng(1)
    samples = [(int(rng.integers(w.num_requests)), int(rng.integers(w.num_q_heads)), int(a))
               for a in list(rng.integers(0, 1280, 60)) + [0, 127, 128, 1023, 1024, 1279]]
    qd, kd, vd = c.host()
    ref, ref_lse = oracle.attend_full_rows(w.full_row_off, w.full_lens, qd, kd, vd, w.softmax_scale, samples)
    got = workloads.to_f64(out)
    got_rows = np.stack([got[w.full_row_off[i] + a, h] for i, h, a in samples])
    check(got_rows, ref, w.dtype, "config2 attend_full sampled")
    c.close()


@pytest.mark.parametrize("name,kw", [
    ("config3", dict(num_layers=2, max_requests=6, prefix_div=8, suffix_div=2)),
    ("config4", dict(num_layers=2, max_requests=12, prefix_div=8, suffix_div=4)),
    ("config5", dict(num_layers=1, max_requests=2, prefix_div=16, suffix_div=8)),
])
def test_scaled_down_configs_elementwise(name, kw):
    w = workloads.scaled_down(workloads.CONFIGS[name](), **kw)
    c = Case(w)
    for lp in range(w.num_layers):
        c.compare_all(lp)
    c.close()


def test_tensor_path_agrees_with_simt_path():
    """On-device cross-check over full tensors: both kernel families see the same pool."""
    w = tiny("cross", 1, 8, 4, 128, torch.bfloat16, [300], [0, 0], [260, 50])
    c = Case(w)
    a, la = c.run_attend(0)
    c.bc.set_path(binding.PATH_SIMT)
    b, lb = c.run_attend(0)
    rows = np.concatenate([np.arange(o, o + n) for o, n in zip(w.suffix_row_off, w.suffix_lens)])
    d = np.abs(workloads.to_f64(a)[rows] - workloads.to_f64(b)[rows])
    assert d.max() <= 2e-2 and d.mean() <= 2e-3
    assert np.abs(workloads.to_f64(la)[rows] - workloads.to_f64(lb)[rows]).max() <= 1e-3
    c.close()
