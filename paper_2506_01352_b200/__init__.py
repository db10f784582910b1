"""B200-native TAH-Quant boundary codec (encode / decode of pipeline-stage boundary tensors)."""
