"""Seeded synthetic inputs shaped like the paper's workloads.

Input generation only -- none of the method's arithmetic lives here.  The paper's
experiments use bf16 gradient vectors of Llama-family decoders trained on C4; neither
the dataset nor the models are available, so these generators reproduce the *shape* of
those inputs (flat parameter vector in declaration order, per-tensor noise scale, K
worker buffers that share a mean) and stand in for them.  Everything is drawn from a
seeded ``torch.Generator`` on the requested device.
"""
import math

import torch

_CHUNK = 1 << 24  # elements generated per temporary


def gpt2_small_tensor_sizes():
    """GPT-2 small (12 layers, d_model 768, MLP 3072, vocab 50257, context 1024), tensors in
    declaration order: 148 tensors, 124,439,808 parameters."""
    dm, ff, vocab, ctx, layers = 768, 3072, 50257, 1024, 12
    sizes = [vocab * dm, ctx * dm]
    for _ in range(layers):
        sizes += [dm, dm,                    # ln_1 weight, bias
                  dm * 3 * dm, 3 * dm,       # attention qkv weight, bias
                  dm * dm, dm,               # attention output projection weight, bias
                  dm, dm,                    # ln_2 weight, bias
                  dm * ff, ff,               # mlp up weight, bias
                  ff * dm, dm]               # mlp down weight, bias
    sizes += [dm, dm]                        # final layer norm
    return sizes


def llama_1b_tensor_sizes():
    """Llama-style decoder: 16 layers, hidden 2048, FFN 8192, 32 query / 8 KV heads (head dim
    64), vocab 128256, tied embeddings: 1,235,814,400 parameters."""
    h, ff, vocab, layers, kv = 2048, 8192, 128256, 16, 8 * 64
    sizes = [vocab * h]
    for _ in range(layers):
        sizes += [h * h, kv * h, kv * h, h * h,  # q, k, v, o
                  h * ff, h * ff, ff * h,        # gate, up, down
                  h, h]                          # two RMS norms
    sizes += [h]
    return sizes


def pseudo_tensor_sizes(d, tensor_elems=1 << 20):
    """A flat vector of d elements cut into 1M-element pseudo tensors (last one ragged)."""
    n_full, rem = divmod(d, tensor_elems)
    return [tensor_elems] * n_full + ([rem] if rem else [])


def equal_shard_offsets(d, n_shards):
    """n_shards contiguous shards; the first d % n_shards shards hold one extra element."""
    q, r = divmod(d, n_shards)
    offs = [0]
    for s in range(n_shards):
        offs.append(offs[-1] + q + (1 if s < r else 0))
    return offs


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def per_tensor_sigma(sizes, seed, lo=0.01, hi=0.2):
    """One noise scale per tensor, log-uniform in [lo, hi] (CPU generator: tiny)."""
    g = _gen(seed, "cpu")
    u = torch.rand(len(sizes), generator=g, dtype=torch.float64)
    return torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo))).tolist()


def _noise_into(out, gen, noise):
    """Fills fp32 `out` with unit-scale noise: standard normal, or Student-t with 3 d.o.f."""
    if noise == "normal":
        out.normal_(generator=gen)
        return
    if noise != "student_t3":
        raise ValueError(noise)
    out.normal_(generator=gen)
    chi2 = torch.zeros_like(out)
    tmp = torch.empty_like(out)
    for _ in range(3):
        tmp.normal_(generator=gen)
        chi2.addcmul_(tmp, tmp)
    out.div_(torch.sqrt(chi2 / 3.0))


def worker_grads(sizes, K, dtype, seed, device, sigma=0.05, mu_std=0.01, noise="normal"):
    """K gradient buffers g_k = mu + sigma_t * xi_k over the flat vector of sum(sizes)
    elements.  mu ~ N(0, mu_std^2) is shared by the workers; xi_k is unit noise, i.i.d. per
    worker; sigma is a float or one value per tensor.  Returns a list of K tensors."""
    d = int(sum(sizes))
    gen = _gen(seed, device)
    per_tensor = not isinstance(sigma, (int, float))
    if per_tensor:
        assert len(sigma) == len(sizes)
    grads = [torch.empty(d, dtype=dtype, device=device) for _ in range(K)]
    bounds = [0]
    for s in sizes:
        bounds.append(bounds[-1] + int(s))
    for c0 in range(0, d, _CHUNK):
        c1 = min(d, c0 + _CHUNK)
        n = c1 - c0
        mu = torch.empty(n, dtype=torch.float32, device=device).normal_(generator=gen) * mu_std
        if per_tensor:
            sig = torch.empty(n, dtype=torch.float32, device=device)
            for t, s_t in enumerate(sigma):  # tensors overlapping [c0, c1)
                lo, hi = max(bounds[t], c0), min(bounds[t + 1], c1)
                if lo < hi:
                    sig[lo - c0:hi - c0] = float(s_t)
        xi = torch.empty(n, dtype=torch.float32, device=device)
        for k in range(K):
            _noise_into(xi, gen, noise)
            if per_tensor:
                xi.mul_(sig)
            else:
                xi.mul_(float(sigma))
            xi.add_(mu)
            grads[k][c0:c1] = xi.to(dtype)
    return grads


def adam_state(d, seed, device, zero_moments=True, param_std=0.02):
    """fp32 master params ~ N(0, param_std^2) and the two AdamW moments: zeros (the state
    Algorithm 1 starts from) or a mid-training state (m small and signed, v positive)."""
    gen = _gen(seed, device)
    p = torch.empty(d, dtype=torch.float32, device=device)
    for c0 in range(0, d, _CHUNK):
        p[c0:c0 + _CHUNK].normal_(generator=gen)
    p.mul_(param_std)
    if zero_moments:
        m = torch.zeros(d, dtype=torch.float32, device=device)
        v = torch.zeros(d, dtype=torch.float32, device=device)
    else:
        m = torch.empty(d, dtype=torch.float32, device=device)
        v = torch.empty(d, dtype=torch.float32, device=device)
        for c0 in range(0, d, _CHUNK):
            m[c0:c0 + _CHUNK].normal_(generator=gen)
            v[c0:c0 + _CHUNK].uniform_(0.25, 1.0, generator=gen)
        m.mul_(0.01)
        v.mul_(0.02 * 0.02)
    return p, m, v


# ---- per-sample workload: linear least squares ------------------------------------------
def lsq_problem(d, seed, device):
    """w* and w0, independent N(0, 1/d)."""
    gen = _gen(seed, device)
    w_star = torch.empty(d, dtype=torch.float32, device=device).normal_(generator=gen) / math.sqrt(d)
    w0 = torch.empty(d, dtype=torch.float32, device=device).normal_(generator=gen) / math.sqrt(d)
    return w_star, w0


def lsq_batch(b, w_star, seed, t):
    """A fresh batch for step t: x ~ N(0, I) [b, d], y = x.w* + 0.1 eps."""
    d, device = w_star.numel(), w_star.device
    gen = _gen(int(seed) * 1000003 + int(t), device)
    x = torch.empty(b, d, dtype=torch.float32, device=device).normal_(generator=gen)
    eps = torch.empty(b, dtype=torch.float32, device=device).normal_(generator=gen)
    y = x @ w_star + 0.1 * eps
    return x, y


def lsq_persample_grads(x, y, w):
    """The model's backward pass for 0.5 (x.w - y)^2: row i = (x_i.w - y_i) x_i, fp32 [b, d]."""
    r = x @ w - y
    return (r[:, None] * x).contiguous()
