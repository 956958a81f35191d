"""Shapes and rates of the synthetic workload configurations.  Plain numbers only: this module imports
nothing, so that code which must not load the CUDA library (the CPU baseline of the benchmark) can read the
same configuration as the code that does."""

MLP_A = [512, 512, 512, 512, 10]
MLP_B = [256, 1024, 256]
VIT_S = dict(d=384, n_layers=12, n_heads=6, mlp=1536, n_cls=1000)
VIT_B = dict(d=768, n_layers=12, n_heads=12, mlp=3072, n_cls=1000)
DEC_1B = dict(d=2048, n_layers=16, n_q_heads=32, n_kv_heads=8, head_dim=64, ffn=8192, vocab=32000)
DEC_8B = dict(d=4096, n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=32000)

# mixed co-resident step: per family the first instance is latency-sensitive, the others frequency-sensitive
MIXED_LS_BATCH, MIXED_FS_BATCH = 4, 256
MIXED_KV_LO, MIXED_KV_HI = 128, 4096
# arrival rates (requests/s) of the 8 instances, fixed table
MIXED_RATES = {"mlp": [2000.0, 1500.0, 1000.0], "vit": [500.0, 300.0, 200.0], "decoder": [100.0, 50.0]}
LS_DEADLINE_NS = 20_000_000

# stress step
STRESS_VITS, STRESS_VIT_BATCH, STRESS_DEC_BATCH = 16, 32, 256
STRESS_KV_LO, STRESS_KV_HI = 512, 8192


def mixed_counts(ls: int = MIXED_LS_BATCH, fs: int = MIXED_FS_BATCH):
    """Requests per family in one saturated mixed step (3 MLP-A, 3 ViT-S, 2 decoders)."""
    return {"mlp": ls + 2 * fs, "vit": ls + 2 * fs, "decoder": ls + fs}
