"""Size accounting of GRASS state (test infrastructure, CPU only).

Restates the paper's memory model (summary table of Section 2: optimizer
2r + 2nr floats, gradient nr floats per m x n weight; Appendix "Experiments:
Pretraining Memory") for a LLaMA-shaped model so that the printed 13B worked
example can serve as a pin of the r x n state sizes the CUDA path allocates.

Readings needed to reproduce the printed figures: "MB" is 2^20 bytes; the
projection acts on the smaller of a weight's two dimensions, so the projected
gradient of an (m x n) weight holds r * max(m, n) numbers; embeddings, LM head
and norm weights keep full gradients and full Adam moments; the cross-entropy
activation term reproduces the printed activation figure only with its fp32
part (B*L*V*4) alone, although the printed formula also lists B*L*V*2.
"""
from __future__ import annotations

MIB = float(2 ** 20)


def llama_weight_shapes(hidden, ffn, layers):
    """(m, n) of every projected linear weight: 4 attention + 3 MLP per layer."""
    per_layer = [(hidden, hidden)] * 4 + [(ffn, hidden)] * 2 + [(hidden, ffn)]
    return per_layer * layers


def grass_memory_mib(hidden, ffn, layers, heads, vocab, seq, batch, r, bytes_per=2):
    shapes = llama_weight_shapes(hidden, ffn, layers)
    unprojected = 2 * vocab * hidden + layers * 2 * hidden + hidden   # embed, head, norms
    n_params = sum(m * n for m, n in shapes) + unprojected

    projected = sum(r * max(m, n) for m, n in shapes)                  # sum of n*r
    gradient = (projected + unprojected) * bytes_per
    optimizer = (2 * projected + 2 * r * len(shapes) + 2 * unprojected) * bytes_per
    parameter = n_params * bytes_per
    extra = vocab * hidden * bytes_per                                 # largest tensor

    emb = batch * seq * hidden
    ln = emb * 2
    attn = ln + emb * 2 + 2 * emb * 2 + batch * heads * seq * seq * 2 \
        + (batch * heads * seq * seq + emb * 2) + emb * 2
    ffwd = ln + emb * 2 + emb * 4 * 2 + emb * 4 * 2
    activation = ln + layers * (attn + ffwd) + emb * 2 + batch * seq * vocab * 4

    out = dict(activation=activation / MIB, parameter=parameter / MIB,
               gradient=gradient / MIB, optimizer=optimizer / MIB, extra=extra / MIB)
    out["total"] = sum(out.values())
    return out
