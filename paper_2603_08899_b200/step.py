"""One verification step = L x confu_tree_attention + confu_tree_accept + confu_kv_compact, enqueued
on one stream through the C-ABI binding.  This module only owns buffers and call order; all
arithmetic runs in the CUDA library."""
import torch

from . import binding as cb


class VerifyStep:
    def __init__(self, cfg, n_slots, device="cuda", ctx=None):
        self.cfg = cfg
        self.n_slots = n_slots
        self.dev = device
        self.own_ctx = ctx is None
        self.ctx = cb.confu_create(torch.device(device).index or 0) if ctx is None else ctx
        self.dims = cb.make_dims(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T, cfg.C, cfg.S, cfg.kv_dtype)
        B, T = cfg.B, cfg.T
        u8 = dict(dtype=torch.uint8, device=device)
        i32 = dict(dtype=torch.int32, device=device)
        self.ws = torch.empty(cb.confu_workspace_bytes(self.ctx, self.dims), **u8)
        cb.confu_set_workspace(self.ctx, self.ws)
        self.plan = torch.empty(cb.confu_plan_bytes(self.ctx, self.dims), **u8)
        self.accept_ws = torch.empty(cb.confu_accept_workspace_bytes(B, T, cfg.V), **u8)
        self.status = torch.zeros(B, **i32)
        self.accept_len = torch.zeros(B, **i32)
        self.path = torch.zeros(B, cb.MAX_DEPTH + 1, **i32)
        self.next_token = torch.zeros(B, **i32)
        self.future_row = torch.zeros(B, **i32)
        self.counters = torch.zeros(B, 4, **i32)
        self.new_prefix_len = torch.zeros(B, **i32)

    def close(self):
        if self.own_ctx:
            cb.confu_destroy(self.ctx)
            self.own_ctx = False

    def bind(self, q_layers, k_layers, v_layers, k_soft, v_soft, out_layers, seq_start, prefix_len, parent,
             con_owner, target_logits, draft_logits, tokens, uniforms, kv_scales=None):
        """Remember the (device) tensors of a step; lists have one entry per layer.  kv_scales: for an
        E4M3 cache, one (k_scale, v_scale) pair of fp32 [Hkv] tensors per layer."""
        self.kv_scales = kv_scales
        self.q, self.k, self.v, self.ks, self.vs, self.out = q_layers, k_layers, v_layers, k_soft, v_soft, out_layers
        self.seq_start, self.prefix_len, self.parent, self.con_owner = seq_start, prefix_len, parent, con_owner
        self.tl, self.dl, self.tokens, self.uniforms = target_logits, draft_logits, tokens, uniforms
        self.k_ptrs = torch.tensor([t.data_ptr() for t in k_layers], dtype=torch.int64, device=self.dev)
        self.v_ptrs = torch.tensor([t.data_ptr() for t in v_layers], dtype=torch.int64, device=self.dev)

    def run_attention(self, lse_layers=None):
        cfg = self.cfg
        cb.confu_tree_plan(self.ctx, self.dims, self.seq_start, self.prefix_len, self.parent, self.con_owner,
                           self.plan, self.status)
        for l in range(len(self.q)):
            if self.kv_scales is not None:
                cb.confu_set_kv_scales(self.ctx, *self.kv_scales[l])
            cb.confu_tree_attention(self.ctx, self.dims, self.q[l], self.k[l], self.v[l], self.n_slots,
                                    self.seq_start, self.prefix_len,
                                    self.ks[l] if self.ks is not None else None,
                                    self.vs[l] if self.vs is not None else None,
                                    None, None, self.plan, self.out[l],
                                    None if lse_layers is None else lse_layers[l], self.status)

    def run_plan(self):
        cb.confu_tree_plan(self.ctx, self.dims, self.seq_start, self.prefix_len, self.parent, self.con_owner,
                           self.plan, self.status)

    def run_layers(self):
        """The L attention calls with the plan built by run_plan()."""
        for l in range(len(self.q)):
            if self.kv_scales is not None:
                cb.confu_set_kv_scales(self.ctx, *self.kv_scales[l])
            cb.confu_tree_attention(self.ctx, self.dims, self.q[l], self.k[l], self.v[l], self.n_slots,
                                    self.seq_start, self.prefix_len,
                                    self.ks[l] if self.ks is not None else None,
                                    self.vs[l] if self.vs is not None else None,
                                    None, None, self.plan, self.out[l], None, self.status)

    def capture(self, temperature=1.0, sibling_mode=1):
        """Record the step's launches once as four CUDA graphs (plan | attention layers | acceptance |
        compaction) over the bound tensors, and once more as a single graph; replay() then enqueues a
        step with four graph launches (events can go between the parts), replay_step() with one,
        instead of 2 L + 4 kernel launches from the host.  Run the step once before capturing (the
        first call of each kernel sets function attributes, which a capture does not allow)."""
        parts = (self.run_plan, self.run_layers, lambda: self.run_accept(temperature, sibling_mode), self.run_compact)
        self.graphs = []
        for fn in parts:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            self.graphs.append(g)
        # and the whole step as one graph: one launch from the host per step (replay_step)
        self.graph_step = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_step):
            for fn in parts:
                fn()

    def replay_step(self):
        """Enqueue one captured step on the current stream as a single graph launch."""
        self.graph_step.replay()

    def replay(self, events=None):
        """Enqueue one captured step on the current stream; events: optional 5 CUDA events recorded
        before the first graph and after each of the four."""
        if events is not None:
            events[0].record()
        for i, g in enumerate(self.graphs):
            g.replay()
            if events is not None:
                events[i + 1].record()

    def run_accept(self, temperature, sibling_mode=1):
        cfg = self.cfg
        cb.confu_tree_accept(self.ctx, cfg.B, cfg.T, cfg.C, cfg.V, cfg.logit_dtype, self.tl,
                             self.dl if temperature > 0 else None, self.tokens, self.parent, self.con_owner,
                             self.uniforms if temperature > 0 else None, temperature, sibling_mode, self.accept_len,
                             self.path, self.next_token, self.future_row, self.counters, self.accept_ws, self.status)

    def run_compact(self):
        cb.confu_kv_compact(self.ctx, self.dims, len(self.k), self.k_ptrs, self.v_ptrs, self.seq_start,
                            self.prefix_len, self.accept_len, self.path, self.new_prefix_len, self.status)

    def run(self, temperature=1.0, sibling_mode=1):
        """The whole step on the current stream (no host synchronisation)."""
        self.run_attention()
        self.run_accept(temperature, sibling_mode)
        self.run_compact()

    def launches_per_step(self):
        """Kernels of this library launched by run(): plan + per layer attention + row statistics +
        walk + compaction."""
        return 1 + self.attention_kernels_per_layer() * len(self.q) + 3

    def attention_path(self):
        """The library's choice of attention kernel for this step's dims (a binding.ATTENTION_* value)."""
        return cb.confu_attention_path(self.ctx, self.dims)

    def attention_kernel_name(self):
        path = self.attention_path()
        if path == cb.ATTENTION_GENERIC:
            return "attention_generic_kernel"
        if path == cb.ATTENTION_TENSOR_PAIR:
            return "attention_pair_kernel"
        return "attention_fp8_kernel" if self.cfg.kv_dtype == torch.float8_e4m3fn else "attention_tc_kernel"

    def attention_kernels_per_layer(self):
        """The tensor-core kernels are followed by the merge of the split pairs; the generic path is one kernel."""
        return 2 if self.attention_path() in (cb.ATTENTION_TENSOR, cb.ATTENTION_TENSOR_PAIR) else 1


def sm_count(step):
    """SM count of the step's device (one attention CTA per SM)."""
    return torch.cuda.get_device_properties(torch.device(step.dev)).multi_processor_count
