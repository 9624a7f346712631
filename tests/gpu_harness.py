"""Plumbing for the GPU parity tests: device buffers via torch, calls through the C ABI binding."""
import numpy as np

CANARY = 0x7FC0  # bf16 NaN: any output row the library fails to write stays NaN


def to_dev(a, dev):
    import torch
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(dev)
    return torch.from_numpy(a).to(dev)


def bf16_dev_to_f32(t):
    """int16/bf16 device tensor -> float32 NumPy (exact)."""
    import torch
    if t.dtype == torch.int16:
        t = t.view(torch.bfloat16)
    return t.float().cpu().numpy()


class Runner:
    """One handle + workspace for one shape; run() executes plan + decode on the current stream."""

    def __init__(self, binding, Hq, Hkv, d, num_pages, max_batch, ld, layout="HND", plan=None, sm_scale=0.0,
                 variant=None, fused=None, page_size=16):
        import torch
        self.torch = torch
        self.dev = torch.device("cuda:0")
        strides = (0, 0, 0)
        if layout == "NHD":
            strides = (page_size * Hkv * d, d, Hkv * d)
        self.h = binding.Handle(Hq, Hkv, d, num_pages, max_batch, ld, page_size=page_size, kv_strides=strides,
                                sm_scale=sm_scale, plan=plan)
        if variant is not None:
            self.h.set_variant(*variant)
        if fused is not None:
            self.h.set_combine_mode(fused)
        self.ws = torch.empty(self.h.workspace_size(), dtype=torch.uint8, device=self.dev)
        self.shape = (Hq, d)

    def run(self, q, k, v, bt, lens, lens_dev=None, check=True):
        """q/k/v/bt: device tensors (int16 or bf16 / int32); lens: host int32 array. Returns device out (int16)."""
        torch = self.torch
        B = int(len(lens))
        out = torch.full((B,) + self.shape, CANARY, dtype=torch.int16, device=self.dev).view(torch.int16)
        if lens_dev is None:
            lens_dev = torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).to(self.dev)
        st = torch.cuda.current_stream().cuda_stream
        self.h.plan(np.asarray(lens, dtype=np.int32), self.ws.data_ptr(), self.ws.numel(), st)
        self.h.decode_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), bt.data_ptr(), lens_dev.data_ptr(),
                           out.data_ptr(), st)
        torch.cuda.synchronize()
        if check:
            assert self.h.debug_error_word() == 0
        return out


def run_host_case(binding, q, k, v, bt, lens, layout="HND", plan=None, sm_scale=0.0, variant=None, fused=None):
    page_size = k.shape[2]
    """Host uint16 inputs (HND order; transposed here for NHD) -> float32 output [B, Hq, d]."""
    import torch
    dev = torch.device("cuda:0")
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    if layout == "NHD":
        k = np.ascontiguousarray(k.transpose(0, 2, 1, 3))
        v = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    r = Runner(binding, Hq, Hkv, d, k.shape[0], max(B, 1), bt.shape[1], layout, plan, sm_scale, variant, fused, page_size)
    out = r.run(to_dev(q, dev), to_dev(k, dev), to_dev(v, dev), to_dev(bt, dev), lens)
    res = bf16_dev_to_f32(out)
    r.h.close()
    return res


def gather_for_oracle(k_dev, v_dev, block_table, seq_lens, rows):
    """Copy the pages of sequences `rows` back to the host as a compact pool and a remapped block
    table, so that the CPU oracle can evaluate sequences of a workload whose pools live on the GPU."""
    import torch
    ids = []
    new_bt = np.full((len(rows), block_table.shape[1]), -1, dtype=np.int32)
    for i, b in enumerate(rows):
        n = (int(seq_lens[b]) + 15) // 16
        new_bt[i, :n] = np.arange(len(ids), len(ids) + n)
        ids.extend(int(x) for x in block_table[b, :n])
    idx = torch.tensor(ids, dtype=torch.long, device=k_dev.device)
    if k_dev.dtype == torch.uint8:   # an 8-bit cache: the codes as they are
        k, v = k_dev[idx].cpu().numpy(), v_dev[idx].cpu().numpy()
    else:
        k = k_dev.view(torch.int16)[idx].cpu().numpy().view(np.uint16)
        v = v_dev.view(torch.int16)[idx].cpu().numpy().view(np.uint16)
    return k, v, new_bt, np.asarray([seq_lens[b] for b in rows], dtype=np.int32)


def row_groups(seq_lens, max_tokens=65536):
    """Every sequence of a batch, in batch order, cut into groups of at most `max_tokens` cached tokens (a
    sequence longer than that is a group of its own): bounds the host memory of one oracle call."""
    groups, cur, tok = [], [], 0
    for b, L in enumerate(int(x) for x in seq_lens):
        if cur and tok + L > max_tokens:
            groups.append(cur)
            cur, tok = [], 0
        cur.append(b)
        tok += L
    if cur:
        groups.append(cur)
    return groups


def compare_every_sequence(got, q_dev, k_dev, v_dev, block_table, seq_lens, oracle_fn, gates, max_tokens=65536):
    """Compares `got` (float array, first axis = sequence) with the oracle on EVERY sequence of the batch: the pages
    of one group of sequences at a time are copied back from the device pools and `oracle_fn(q, k, v, bt, lens)`
    is evaluated on them.  Asserts both gates element-wise; returns (max abs err, worst tight-gate ratio)."""
    import torch
    worst_abs, worst_ratio, checked = 0.0, 0.0, 0
    for rows in row_groups(seq_lens, max_tokens):
        kh, vh, bth, lh = gather_for_oracle(k_dev, v_dev, block_table, seq_lens, rows)
        qh = q_dev.view(torch.int16)[rows[0]:rows[-1] + 1].cpu().numpy().view(np.uint16)
        ref = oracle_fn(qh, kh, vh, bth, lh)
        g = got[rows[0]:rows[-1] + 1]
        assert gates.stated_violations(g, ref) == 0, (rows[0], rows[-1])
        assert gates.tight_violations(g, ref) == 0, (rows[0], rows[-1], gates.tight_ratio(g, ref))
        worst_abs = max(worst_abs, float(np.max(np.abs(g - ref))) if g.size else 0.0)
        worst_ratio = max(worst_ratio, gates.tight_ratio(g, ref))
        checked += len(rows)
    assert checked == len(seq_lens)
    return worst_abs, worst_ratio
